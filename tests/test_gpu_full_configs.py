"""GPU parity at the full sizes of the benchmark's configurations, in the launch configuration that
bench.py times (deferred error-feedback subtraction on, theta_local buffers shared through shifted
views for the 2B case).  The CUDA path runs on the whole model; the oracle recomputes a sample of tensors
(one of every kind: blocked matrices, norm vectors shorter than a chunk, the flat-path router,
experts with exactly zero drift) from copies taken before the step.  Bars as everywhere: payload
bytes and error buffers bit-exact, theta_sync within 1e-6 x RMS of the tensor."""
import gc

import pytest
import torch

from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _case(wl, **kw):
    from parity import DeviceCase, oracle_threads
    gc.collect()
    torch.cuda.empty_cache()
    oracle_threads()
    c = DeviceCase(wl, **kw)
    c.sl.set_ef_deferred(True)
    return c


def _ids(wl, names):
    from parity import sample_tensor_ids
    ids = sample_tensor_ids(wl, names)
    assert len(ids) == len(names), "sample names must exist in the workload"
    return ids


def _run(c, ids, steps):
    for step in range(steps):
        c.fill_local(step)
        snap = c.snapshot(ids)
        c.step()
        rep = c.check(snap)
        assert rep["tensors"] == len(ids)
    return rep


def test_config2_dense_d768_three_steps():
    wl = I.workload("c2_dense_d768")
    c = _case(wl)
    assert c.sl.payload_bytes() == 4445152
    _run(c, _ids(wl, ["l0.q", "l5.gate", "l11.down", "l3.norm1", "final_norm"]), steps=3)


@pytest.mark.parametrize("k", [41, 82, 123])
def test_config3_dense_d1280_k_sweep(k):
    wl = I.workload("c3_dense_d1280")
    c = _case(wl, k=k)
    assert c.sl.payload_bytes() == {41: 13895424, 82: 25008960, 123: 38900880}[k]
    _run(c, _ids(wl, ["l0.k", "l12.up", "l23.down", "l7.norm2"]), steps=2)


def test_config4_moe_zero_experts_two_steps():
    wl = I.workload("c4_moe_d1024")
    c = _case(wl)
    assert c.sl.payload_bytes() == 19694816
    names = ["l0.router", "l0.o", "l11.norm1"] + [f"l2.x{x}.gate" for x in range(8)] + ["l5.x3.down", "l5.x6.down"]
    _run(c, _ids(wl, names), steps=2)


def test_config5_dense_d2048_as_benchmarked():
    """The benchmark's launch configuration: R = 16, 8 theta_local buffers shared through views shifted by
    2^26 elements, deferred subtraction, seeded non-zero error buffers.  The oracle recomputes 8 of the
    219 tensors: one of every shape class, among them the 32000 x 2048 embedding (16,000 chunks, 250
    summation groups per worker) and an 8192 x 2048 feed-forward matrix; the CUDA path runs all 219."""
    import numpy as np
    from bench import ALIAS_SHIFT
    wl = I.workload("c5_dense_d2048")
    c = _case(wl, distinct_local=8, e_scale=0.5, alias_shift=ALIAS_SHIFT)
    assert c.sl.payload_bytes() == 47633184
    ids = _ids(wl, ["embed", "l0.q", "l5.gate", "l9.v", "l23.down", "l17.norm1", "final_norm", "l12.up"])
    assert len(wl.tensors) == 219
    for step in range(2):
        c.fill_local(step)
        # Reading the true error while corrected values wait in the workspace needs one flat spare buffer,
        # and 25 model-sized buffers leave no room for a 26th: the first theta_local buffer serves (the
        # snapshot copies the parameters before it uses the spare) and is refilled before the step; after
        # the step theta_local is not needed any more.
        snap = c.snapshot(ids, spare=c.local[0])
        I.theta_local(wl, c.theta, 0, step, out=c.local[0])
        c.step()
        rep = c.check(snap, spare=c.local[0])
        assert rep["tensors"] == len(ids)
    # the waiting values can be written out and leave the true error in the buffers themselves
    want = c.error_slices(ids[:2], spare=c.local[0])
    c.sl.ef_flush()
    torch.cuda.synchronize()
    assert not c.sl.ef_pending()
    got = c.error_slices(ids[:2])
    for r in range(wl.R):
        for j in ids[:2]:
            assert np.array_equal(got[r][j].view(np.uint32), want[r][j].view(np.uint32))
    assert c.guards_intact()


def test_repeated_runs_leave_identical_bits():
    """The same three steps from the same state on two independent sets of buffers: theta, every error
    buffer, every payload and the values waiting in the workspace must agree bit for bit, whatever the
    scheduling of warps and CTAs was (the ordered additions of Eq. 2 line 3, the deterministic candidate
    lists and tie rule of the selection).  Run on the 162 M-parameter config, where every kernel spans
    many waves."""
    wl = I.workload("c2_dense_d768")
    a = _case(wl, e_scale=0.5)
    b = _case(wl, e_scale=0.5)
    for step in range(3):
        a.fill_local(step)
        b.fill_local(step)
        a.step()
        b.step()
        torch.cuda.synchronize()
        assert torch.equal(a.theta.view(torch.int32), b.theta.view(torch.int32)), step
        for r in range(wl.R):
            assert torch.equal(a.payloads[r], b.payloads[r]), (step, r)
            assert torch.equal(a.e[r].view(torch.int32), b.e[r].view(torch.int32)), (step, r)
    ea, eb = a.true_error(), b.true_error()
    for r in range(wl.R):
        assert torch.equal(ea[r].view(torch.int32), eb[r].view(torch.int32)), r
