"""Pins for the oracle's dense baselines: DiLoCo's outer step (Eq. 1) against a direct numpy
evaluation and its special cases, and Proposition 1 (DiLoCo-LOM with equal initial momenta takes the
same steps as DiLoCo with a global momentum) between two separately written routines."""
import numpy as np

import oracle as O


def _setup(seed, R=4, shapes=((8, 12), (1, 37), (64, 64))):
    rng = np.random.default_rng(seed)
    tab = O.Table(shapes, offsets=[0, 100, 140])   # gaps between tensors must stay untouched
    n = tab.numel
    theta = rng.standard_normal(n).astype(np.float32)
    theta_r = [(theta - 0.01 * rng.standard_normal(n)).astype(np.float32) for _ in range(R)]
    return tab, theta, theta_r, n, rng


def _mask(tab, n):
    mk = np.zeros(n, bool)
    for r, c, o in tab.shapes:
        mk[o:o + r * c] = True
    return mk


def test_diloco_step_against_numpy_and_gaps_untouched():
    tab, theta, theta_r, n, rng = _setup(1)
    m = (0.1 * rng.standard_normal(n)).astype(np.float32)
    t0, m0 = theta.copy(), m.copy()
    O.diloco_step(tab, theta, theta_r, m, 0.9, 0.7)
    mk = _mask(tab, n)
    dbar = np.mean([t0.astype(np.float64) - x.astype(np.float64) for x in theta_r], axis=0)
    mm = 0.9 * m0.astype(np.float64) + dbar          # 0.9, 0.7 as fp32 differ from these doubles by 1e-8 relative
    want = t0.astype(np.float64) - 0.7 * (dbar + 0.9 * mm)
    assert np.allclose(theta[mk], want[mk], rtol=0, atol=1e-6)
    assert np.allclose(m[mk], mm[mk], rtol=0, atol=1e-7)
    assert np.array_equal(theta[~mk], t0[~mk]) and np.array_equal(m[~mk], m0[~mk])


def test_diloco_special_cases():
    tab, theta, theta_r, n, rng = _setup(2, R=3)
    mk = _mask(tab, n)
    # beta = 0, alpha = 1: plain parameter averaging
    m = np.zeros(n, np.float32)
    t = theta.copy()
    O.diloco_step(tab, t, theta_r, m, 0.0, 1.0)
    avg = np.mean([x.astype(np.float64) for x in theta_r], axis=0)
    assert np.allclose(t[mk], avg[mk], rtol=0, atol=2e-7)
    # alpha = 0: theta unchanged, momentum still accumulates
    m = np.zeros(n, np.float32)
    t = theta.copy()
    O.diloco_step(tab, t, theta_r, m, 0.5, 0.0)
    assert np.array_equal(t, theta) and np.any(m[mk] != 0)
    # no drift: nothing moves
    m = np.zeros(n, np.float32)
    t = theta.copy()
    O.diloco_step(tab, t, [theta.copy() for _ in range(3)], m, 0.9, 0.7)
    assert np.array_equal(t, theta) and not np.any(m)


def test_proposition_1_local_outer_momentum_equals_global():
    tab, theta, theta_r0, n, rng = _setup(3, R=4)
    th_g, th_l = theta.copy(), theta.copy()
    m = np.zeros(n, np.float32)
    m_r = [np.zeros(n, np.float64) for _ in range(4)]
    for step in range(5):
        # fresh replicas around the current parameters (the same drifts for both methods)
        drift = [0.01 * rng.standard_normal(n) for _ in range(4)]
        O.diloco_step(tab, th_g, [(th_g - d).astype(np.float32) for d in drift], m, 0.9, 0.7)
        O.diloco_lom_step(tab, th_l, [(th_l - d).astype(np.float32) for d in drift], m_r, 0.9, 0.7)
        mk = _mask(tab, n)
        assert np.allclose(th_g[mk], th_l[mk], rtol=0, atol=5e-6), step
        # the mean of the local momenta is the global momentum
        assert np.allclose(np.mean(m_r, axis=0)[mk], m[mk], rtol=0, atol=5e-6)
