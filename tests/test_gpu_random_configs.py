"""Seeded random configurations of the whole outer step against the oracle: tensor tables mixing blocked,
flat, short and tiny tensors, k from 1 to 2048, every quantiser width, 1 to 5 workers, the deferred
subtraction on and off, a frozen step in between (App. "Freezing Error Feedback") and an absent worker
in sl_aggregate_apply.  Bars as everywhere: payload bytes and error buffers bit for bit, theta within
1e-6 x RMS (Eq. 2, Alg. 1).  The cases are drawn from a fixed seed, so a failure names its case."""
import numpy as np
import pytest
import torch

from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu

KS = [1, 2, 3, 17, 41, 64, 100, 128, 129, 200, 256, 257, 300, 700, 1000, 2048]


def _draw(seed: int):
    rng = np.random.default_rng(1000 + seed)
    pool = [lambda: (64 * int(rng.integers(1, 4)), 64 * int(rng.integers(1, 5))),      # blocked
            lambda: (1, int(rng.integers(1, 3)) * 4096 + int(rng.integers(1, 4096))),   # flat with a short tail
            lambda: (1, int(rng.integers(1, 200))),                                     # tiny
            lambda: (int(rng.integers(3, 90)), int(rng.integers(65, 130))),             # 2-D that is not blocked: flat
            lambda: (1, 4096 * int(rng.integers(1, 4)))]                                # flat, whole chunks
    n = int(rng.integers(3, 7))
    tensors = []
    for j in range(n):
        rows, cols = pool[int(rng.integers(0, len(pool)))]()
        tensors.append(I.TensorSpec(f"t{j}", rows, cols, j % 3))
    R = int(rng.choice([1, 2, 3, 5]))
    k = int(rng.choice(KS))
    bits = 2 if rng.random() < 0.5 else int(rng.choice([1, 3, 4]))
    deferred = bool(bits == 2 and k <= 256 and rng.random() < 0.5)
    recipe = str(rng.choice(["normal", "student_t4"]))
    freeze_step = int(rng.integers(0, 3))   # 1: the middle one of the three steps runs with error feedback frozen
    return tensors, R, k, bits, deferred, recipe, freeze_step, float(rng.uniform(0.3, 1.0)), float(rng.uniform(0.0, 1.0))


@pytest.mark.parametrize("seed", range(28))
def test_random_configuration(seed):
    from parity import DeviceCase, oracle_threads
    oracle_threads()
    tensors, R, k, bits, deferred, recipe, freeze_step, lr, beta = _draw(seed)
    wl = I.Workload(f"random{seed}", tensors, R=R, k=k, recipe=recipe, seed=seed, outer_lr=lr, beta=beta)
    c = DeviceCase(wl, e_scale=0.5, quant_bits=bits)
    if deferred:
        c.sl.set_ef_deferred(True)
    ids = range(len(tensors))
    for step in range(3):
        frozen = step == 1 and freeze_step == 1
        c.sl.set_hyper(ef_enabled=not frozen)
        c.fill_local(step)
        snap = c.snapshot(ids)
        c.step()
        rep = c.check(snap, ef_enabled=not frozen)
        assert rep["tensors"] == len(tensors), (seed, R, k, bits, deferred)
    c.sl.set_hyper(ef_enabled=True)
    if R > 1:  # the two halves on their own, the last worker absent
        if deferred:
            c.sl.ef_flush()
            c.sl.set_ef_deferred(False)
        c.fill_local(3)
        snap = c.snapshot(ids)
        for r in range(R):
            c.sl.compress(c.theta, c.local_of(r), c.e[r], c.payloads[r])
        present = [r != R - 1 for r in range(R)]
        c.sl.aggregate_apply([c.payloads[r] if present[r] else None for r in range(R)], c.theta)
        torch.cuda.synchronize()
        assert c.guards_intact()
        c.check(snap, present=present)
