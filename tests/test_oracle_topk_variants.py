"""Pins for the oracle's Top-k / local-momentum variants (App. "Exact algorithmic description of DiLoCo
variants", Alg. 2-4; Sec. 3.2).  Each is checked against something written independently here: a
numpy evaluation with a brute-force chunk-wise Top-k (argsort with the lowest-index tie rule), and the
reductions the paper states -- Alg. 3 with error feedback and no outer momentum is SparseLoCo without
the quantiser; with k = chunk size every variant is its dense counterpart; DiLoCo-LOM takes DiLoCo's
steps (Proposition 1); Sub-k leaves the update alone and zeroes exactly the Top-k of each momentum."""
import numpy as np
import pytest

import oracle as O

C_SMALL, TILE = 16, 4          # small chunks so that brute force is cheap: 4x4 blocks, runs of 16
SHAPES = ((8, 12), (1, 37), (4, 4), (6, 5))   # blocked, flat with a short tail, one block, 2-D but not blockable
OFFS = [0, 100, 140, 160]


def _setup(seed, R, k):
    rng = np.random.default_rng(seed)
    tab = O.Table(SHAPES, offsets=OFFS)
    n = tab.numel
    cfg = O.Config(k=k, R=R, beta=0.9, outer_lr=0.7, chunk_elems=C_SMALL, tile_dim=TILE, quant_bits=32)
    theta = rng.standard_normal(n).astype(np.float32)
    return rng, tab, cfg, theta, n


def _replicas(rng, theta, R):
    return [(theta - 0.05 * rng.standard_normal(theta.size)).astype(np.float32) for _ in range(R)]


def _chunks():
    """Flat positions of every chunk of the table, independently of the oracle's geometry code."""
    out = []
    for (rows, cols), off in zip(SHAPES, OFFS):
        if rows > 1 and rows % TILE == 0 and cols % TILE == 0:
            for a in range(rows // TILE):
                for b in range(cols // TILE):
                    out.append([off + (a * TILE + i) * cols + b * TILE + j for i in range(TILE) for j in range(TILE)])
        else:
            n = rows * cols
            for s in range(0, n, C_SMALL):
                out.append([off + p for p in range(s, min(s + C_SMALL, n))])
    return out


def _topk_positions(u, k):
    """Brute force: per chunk the k largest |u| (bit pattern order = magnitude order for finite values),
    ties to the lower in-chunk index."""
    sel = []
    for ch in _chunks():
        mag = np.abs(u[ch].astype(np.float64))
        order = sorted(range(len(ch)), key=lambda p: (-mag[p], p))[:min(k, len(ch))]
        sel.extend(ch[p] for p in order)
    return np.array(sorted(sel), dtype=np.int64)


def _mask(n):
    mk = np.zeros(n, bool)
    for (r, c), o in zip(SHAPES, OFFS):
        mk[o:o + r * c] = True
    return mk


f32 = np.float32


def _fma(a, b, c):
    """fma(a, b, c) for fp32 arrays, single rounding (exact product and sum in fp64 for these magnitudes
    would double-round in rare cases; the exact value is formed as a rational-free long double sum)."""
    return (np.longdouble(a) * np.longdouble(b) + np.longdouble(c)).astype(np.float32)


@pytest.mark.parametrize("use_ef", [False, True])
def test_alg3_against_numpy_with_brute_force_topk(use_ef):
    rng, tab, cfg, theta, n = _setup(11, R=3, k=5)
    mk = _mask(n)
    m = (0.1 * rng.standard_normal(n)).astype(np.float32) * mk
    e = [(0.02 * rng.standard_normal(n)).astype(np.float32) * mk for _ in range(3)] if use_ef else None
    mu = 0.8
    for step in range(3):
        reps = _replicas(rng, theta, 3)
        t0, m0 = theta.copy(), m.copy()
        e0 = [x.copy() for x in e] if use_ef else None
        O.diloco_topk_step(cfg, tab, theta, reps, e, m, mu)
        acc = np.zeros(n, np.float64)
        for r in range(3):
            d = (t0 - reps[r]).astype(np.float32)
            u = _fma(f32(cfg.beta), e0[r], d) if use_ef else d
            u = u * mk
            sel = _topk_positions(u, cfg.k)
            acc[sel] += u[sel].astype(np.float64)
            if use_ef:
                want_e = u.copy()
                want_e[sel] = 0.0
                assert np.array_equal(e[r][mk], want_e[mk]), (step, r)
        dbar = acc / 3
        mm = np.float64(f32(mu)) * m0.astype(np.float64) + dbar
        want = t0.astype(np.float64) - np.float64(f32(cfg.outer_lr)) * (dbar + np.float64(f32(mu)) * mm)
        assert np.array_equal(theta[mk], want.astype(np.float32)[mk]), step
        assert np.array_equal(m[mk], mm.astype(np.float32)[mk]), step
        assert np.array_equal(theta[~mk], t0[~mk])


@pytest.mark.parametrize("use_ef", [False, True])
def test_alg4_against_numpy_with_brute_force_topk(use_ef):
    rng, tab, cfg, theta, n = _setup(12, R=3, k=4)
    mk = _mask(n)
    m_r = [(0.1 * rng.standard_normal(n)).astype(np.float32) * mk for _ in range(3)]
    e = [(0.02 * rng.standard_normal(n)).astype(np.float32) * mk for _ in range(3)] if use_ef else None
    mu = 0.6
    for step in range(3):
        reps = _replicas(rng, theta, 3)
        t0 = theta.copy()
        m0 = [x.copy() for x in m_r]
        e0 = [x.copy() for x in e] if use_ef else None
        O.lom_topk_step(cfg, tab, theta, reps, m_r, e, mu)
        acc = np.zeros(n, np.float64)
        hit = np.zeros(n, bool)
        for r in range(3):
            d = (t0 - reps[r]).astype(np.float32)
            mm = _fma(f32(mu), m0[r], d)
            nd = _fma(f32(mu), mm, d)
            u = (_fma(f32(cfg.beta), e0[r], nd) if use_ef else nd) * mk
            assert np.array_equal(m_r[r][mk], mm[mk])
            sel = _topk_positions(u, cfg.k)
            acc[sel] += u[sel].astype(np.float64)
            hit[sel] = True
            if use_ef:
                want_e = u.copy()
                want_e[sel] = 0.0
                assert np.array_equal(e[r][mk], want_e[mk])
        want = (t0.astype(np.float64) - np.float64(f32(cfg.outer_lr)) * acc / 3).astype(np.float32)
        assert np.array_equal(theta[hit], want[hit]) and np.array_equal(theta[~hit], t0[~hit])


def test_alg3_with_ef_and_no_momentum_is_sparseloco_without_the_quantiser():
    rng, tab, cfg, theta, n = _setup(13, R=4, k=3)
    th_a, th_b = theta.copy(), theta.copy()
    e_a = [np.zeros(n, np.float32) for _ in range(4)]
    e_b = [np.zeros(n, np.float32) for _ in range(4)]
    m = np.zeros(n, np.float32)
    for step in range(4):
        drift = [0.05 * rng.standard_normal(n) for _ in range(4)]
        O.diloco_topk_step(cfg, tab, th_a, [(th_a - d).astype(np.float32) for d in drift], e_a, m, 0.0)
        # SparseLoCo's own routines with quant_bits = 32 (values travel unquantised): Eq. 2 without Q
        outs = [O.compress(cfg, tab, th_b, (th_b - d).astype(np.float32), e_b[r]) for r, d in enumerate(drift)]
        O.aggregate_apply_sparse(cfg, tab, [o.sel_idx for o in outs], [o.sel_hat for o in outs], th_b)
        assert np.array_equal(th_a, th_b), step
        for r in range(4):
            assert np.array_equal(e_a[r], e_b[r])


def test_k_equal_to_the_chunk_size_gives_the_dense_methods():
    """Top-k with k = C keeps everything: Alg. 3 without EF is DiLoCo (Eq. 1); Alg. 4 without EF is
    DiLoCo-LOM (Alg. 2), which by Proposition 1 takes DiLoCo's steps."""
    rng, tab, cfg, theta, n = _setup(14, R=3, k=C_SMALL)
    mk = _mask(n)
    th3, th4, th2, thd = (theta.copy() for _ in range(4))
    m3, md = np.zeros(n, np.float32), np.zeros(n, np.float32)
    m4 = [np.zeros(n, np.float32) for _ in range(3)]
    m2 = [np.zeros(n, np.float32) for _ in range(3)]
    for step in range(4):
        drift = [0.05 * rng.standard_normal(n) for _ in range(3)]
        O.diloco_topk_step(cfg, tab, th3, [(th3 - d).astype(np.float32) for d in drift], None, m3, 0.9)
        O.lom_topk_step(cfg, tab, th4, [(th4 - d).astype(np.float32) for d in drift], m4, None, 0.9)
        O.lom_step(cfg, tab, th2, [(th2 - d).astype(np.float32) for d in drift], m2, 0.9)
        O.diloco_step(tab, thd, [(thd - d).astype(np.float32) for d in drift], md, 0.9, cfg.outer_lr)
        for got in (th3, th4, th2):
            assert np.allclose(got[mk], thd[mk], rtol=0, atol=2e-6), step
        assert np.allclose(m3[mk], md[mk], rtol=0, atol=2e-6)
        assert np.allclose(np.mean(m4, axis=0)[mk], md[mk], rtol=0, atol=2e-6)   # Proposition 1: mean of local momenta
        assert np.array_equal(th4, th2)                                             # same recipe, nothing dropped


def test_sub_k_zeroes_the_topk_of_each_momentum_and_nothing_else():
    rng, tab, cfg, theta, n = _setup(15, R=3, k=3)
    mk = _mask(n)
    m_a = [(0.1 * rng.standard_normal(n)).astype(np.float32) * mk for _ in range(3)]
    m_b = [x.copy() for x in m_a]
    th_a, th_b = theta.copy(), theta.copy()
    reps = _replicas(rng, theta, 3)
    O.lom_step(cfg, tab, th_a, reps, m_a, 0.9, sub_k=False)
    O.lom_step(cfg, tab, th_b, reps, m_b, 0.9, sub_k=True)
    assert np.array_equal(th_a, th_b)                       # the parameter update does not see the subtraction
    for r in range(3):
        sel = _topk_positions(m_a[r], cfg.k)
        want = m_a[r].copy()
        want[sel] = 0.0
        assert np.array_equal(m_b[r], want)
        assert sel.size == sum(min(cfg.k, len(ch)) for ch in _chunks())
