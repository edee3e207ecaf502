"""GPU parity for the paper's Top-k / local-outer-momentum variants (Sec. 3.2; appendix "Exact algorithmic
description of DiLoCo variants", Alg. 2-4) against the CPU oracle, through the C ABI.  What a worker keeps
(m_r, e_r) is formed by the same single-rounded fp32 operations on both sides and must be bit-exact, and
with it the Top-k selections; theta and the global momentum (fp32 recipe on the GPU, fp64 in the oracle)
within 1e-6 x RMS of the tensor."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu

TENSORS = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 5000, 0), I.TensorSpec("router", 8, 1024, 1),
           I.TensorSpec("norm", 1, 768, 1), I.TensorSpec("tiny", 1, 40, 2), I.TensorSpec("b", 192, 64, 3)]
TOL = 1e-6


def _setup(R, k, seed):
    from paper_2508_15706_b200.binding import SparseLoCo
    O.set_threads(8)
    dev = torch.device("cuda", torch.cuda.current_device())
    wl = I.Workload("variants", TENSORS, R=R, k=k, recipe="student_t4", seed=seed, outer_lr=0.7, beta=0.9)
    shapes, offs = [(t.rows, t.cols) for t in TENSORS], I.offsets(TENSORS)
    sl = SparseLoCo(shapes, offs, k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr)
    cfg = O.Config(k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=32)
    tab = O.Table(shapes, offs)
    theta = I.theta_sync(wl, dev)
    return wl, sl, cfg, tab, theta, dev


def _close(got: torch.Tensor, want: np.ndarray, what, ulps: float = 0.0):
    """Max-abs error within 1e-6 x RMS of the tensor; with `ulps`, plus that many fp32 units in the last
    place of the element (the global momentum is heavy-tailed -- a few selected entries are far above its
    RMS -- and the fp32 recipe rounds it twice per step, the fp64 evaluation once)."""
    offs = I.offsets(TENSORS)
    g = got.cpu().numpy().astype(np.float64)
    for t, off in zip(TENSORS, offs):
        w = want[off:off + t.numel].astype(np.float64)
        rms = float(np.sqrt(np.mean(w ** 2)))
        err = np.abs(g[off:off + t.numel] - w)
        bound = TOL * rms + ulps * 2.0 ** -23 * np.abs(w) + 1e-30
        assert np.all(err <= bound), (what, t.name, float(err.max()), rms)


def _bits_equal(got: torch.Tensor, want: np.ndarray, what):
    assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32)), what


@pytest.mark.parametrize("sub_k", [False, True])
def test_lom_step_alg2(sub_k):
    wl, sl, cfg, tab, theta, dev = _setup(R=3, k=64, seed=61)
    m = [I.initial_error(wl, r, dev, scale=0.3) for r in range(3)]
    th_o, m_o = theta.cpu().numpy().copy(), [x.cpu().numpy().copy() for x in m]
    for step in range(3):
        local = [I.theta_local(wl, theta, r, step) for r in range(3)]
        O.lom_step(cfg, tab, th_o, [(x.cpu().numpy()) for x in local], m_o, 0.9, sub_k=sub_k)
        sl.lom_step(theta, local, m, 0.9, sub_k=sub_k)
        torch.cuda.synchronize()
        assert sl.device_status() == 0
        for r in range(3):
            _bits_equal(m[r], m_o[r], ("m", step, r))
        _close(theta, th_o, ("theta", step))
        theta.copy_(torch.from_numpy(th_o))  # both sides continue from the same parameters


@pytest.mark.parametrize("use_ef,k", [(False, 64), (True, 64), (True, 41), (True, 200)])
def test_diloco_topk_step_alg3(use_ef, k):
    wl, sl, cfg, tab, theta, dev = _setup(R=4, k=k, seed=62)
    e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(4)] if use_ef else None
    mom = I.initial_error(wl, 9, dev, scale=0.2)
    th_o, mom_o = theta.cpu().numpy().copy(), mom.cpu().numpy().copy()
    e_o = [x.cpu().numpy().copy() for x in e] if use_ef else None
    for step in range(3):
        local = [I.theta_local(wl, theta, r, step) for r in range(4)]
        O.diloco_topk_step(cfg, tab, th_o, [x.cpu().numpy() for x in local], e_o, mom_o, 0.8)
        sl.diloco_topk_step(theta, local, e, mom, 0.8)
        torch.cuda.synchronize()
        assert sl.device_status() == 0
        if use_ef:
            for r in range(4):
                _bits_equal(e[r], e_o[r], ("e", step, r))
        _close(theta, th_o, ("theta", step))
        _close(mom, mom_o, ("momentum", step), ulps=2.0)
        theta.copy_(torch.from_numpy(th_o))
        mom.copy_(torch.from_numpy(mom_o))


@pytest.mark.parametrize("use_ef", [False, True])
def test_lom_topk_step_alg4(use_ef):
    wl, sl, cfg, tab, theta, dev = _setup(R=3, k=64, seed=63)
    e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(3)] if use_ef else None
    m = [I.initial_error(wl, 20 + r, dev, scale=0.3) for r in range(3)]
    th_o = theta.cpu().numpy().copy()
    m_o = [x.cpu().numpy().copy() for x in m]
    e_o = [x.cpu().numpy().copy() for x in e] if use_ef else None
    for step in range(3):
        local = [I.theta_local(wl, theta, r, step) for r in range(3)]
        O.lom_topk_step(cfg, tab, th_o, [x.cpu().numpy() for x in local], m_o, e_o, 0.6)
        sl.lom_topk_step(theta, local, m, e, 0.6)   # consumes `local`
        torch.cuda.synchronize()
        assert sl.device_status() == 0
        for r in range(3):
            _bits_equal(m[r], m_o[r], ("m", step, r))
            if use_ef:
                _bits_equal(e[r], e_o[r], ("e", step, r))
        _close(theta, th_o, ("theta", step))
        theta.copy_(torch.from_numpy(th_o))


def test_alg3_with_ef_and_no_momentum_equals_the_outer_step_without_quantiser_on_the_gpu():
    """The reduction the paper's construction rests on, through the library: DiLoCo + Top-k + EF with
    mu = 0 leaves the same error buffers as SparseLoCo's step (whose Top-k selection it shares; the
    quantiser only changes what is sent), i.e. e differs exactly at the selected positions."""
    wl, sl, cfg, tab, theta, dev = _setup(R=2, k=64, seed=64)
    e_a = [I.initial_error(wl, r, dev, scale=0.5) for r in range(2)]
    e_b = [x.clone() for x in e_a]
    local = [I.theta_local(wl, theta, r, 0) for r in range(2)]
    th_a, th_b = theta.clone(), theta.clone()
    mom = torch.zeros_like(theta)
    pay = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(2)]
    sl.diloco_topk_step(th_a, local, e_a, mom, 0.0)
    sl.outer_step(th_b, local, e_b, pay)
    torch.cuda.synchronize()
    chunks, slots = sl.num_chunks()
    for r in range(2):
        differ = (e_a[r].view(torch.int32) != e_b[r].view(torch.int32))
        assert int(differ.sum()) <= slots                  # only selected entries can differ
        assert bool((e_a[r][differ] == 0).all())           # and without a quantiser nothing stays behind there


@pytest.mark.parametrize("ef_enabled", [True, False])
def test_outer_step_without_quantiser(ef_enabled):
    """quant_bits = 32 (the full-precision column of the paper's quantisation ablation): sl_outer_step
    against the oracle's compression with the same setting followed by its sparse aggregation."""
    from paper_2508_15706_b200.binding import SparseLoCo
    wl, _, cfg, tab, theta, dev = _setup(R=3, k=64, seed=65)
    shapes, offs = [(t.rows, t.cols) for t in TENSORS], I.offsets(TENSORS)
    sl = SparseLoCo(shapes, offs, k=64, R=3, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=32, ef_enabled=ef_enabled)
    cfg = O.Config(k=64, R=3, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=32, ef_enabled=int(ef_enabled))
    e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(3)]
    th_o, e_o = theta.cpu().numpy().copy(), [x.cpu().numpy().copy() for x in e]
    for step in range(2):
        local = [I.theta_local(wl, theta, r, step) for r in range(3)]
        outs = [O.compress(cfg, tab, th_o, local[r].cpu().numpy(), e_o[r]) for r in range(3)]
        O.aggregate_apply_sparse(cfg, tab, [o.sel_idx for o in outs], [o.sel_hat for o in outs], th_o)
        sl.outer_step(theta, local, e if ef_enabled else None, [None] * 3)   # no payload format: none is written
        torch.cuda.synchronize()
        assert sl.device_status() == 0
        for r in range(3):
            _bits_equal(e[r], e_o[r], ("e", step, r))
        _close(theta, th_o, ("theta", step))
        theta.copy_(torch.from_numpy(th_o))
    with pytest.raises(Exception):
        sl.compress(theta, local[0], e[0], torch.zeros(64, dtype=torch.uint8, device=dev))


@pytest.mark.parametrize("bits,k", [(1, 64), (3, 64), (4, 64), (3, 41), (4, 123)])
def test_quantiser_widths_of_the_ablation(bits, k):
    """quant_bits 1, 3 and 4 (the paper's quantisation ablation; Sec. 4 defines the quantiser for any
    width): the whole outer step against the oracle -- payload bytes (tables of 2^bits entries, codes of
    `bits` bits) and error buffers bit for bit, theta within 1e-6 x RMS -- over two steps, on blocked,
    flat, short and tiny tensors; and sl_compress + sl_aggregate_apply with an absent worker."""
    from parity import DeviceCase, oracle_threads
    oracle_threads()
    tensors = TENSORS + [I.TensorSpec("wide", 320, 256, 4)]   # 20 chunks... and one of more than 64 chunks below
    tensors = tensors + [I.TensorSpec("big", 576, 512, 5)]
    wl = I.Workload("widths", tensors, R=3, k=k, recipe="student_t4", seed=300 + bits, outer_lr=0.7)
    c = DeviceCase(wl, e_scale=0.5, quant_bits=bits)
    assert c.sl.payload_bytes() == c.payload_bytes
    for step in range(2):
        c.fill_local(step)
        snap = c.snapshot(range(len(tensors)))
        c.step()
        rep = c.check(snap)
        assert rep["tensors"] == len(tensors)
    # the two halves through their own entry points, worker 1 absent
    c.fill_local(2)
    snap = c.snapshot(range(len(tensors)))
    for r in (0, 2):
        c.sl.compress(c.theta, c.local_of(r), c.e[r], c.payloads[r])
    e1 = c.e[1].clone()
    c.sl.aggregate_apply([c.payloads[0], None, c.payloads[2]], c.theta)
    torch.cuda.synchronize()
    assert c.guards_intact()
    c.e[1].copy_(e1)
    cfg = O.Config(k=k, R=3, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=bits)
    for j, t in enumerate(tensors):
        tab = O.Table([(t.rows, t.cols)])
        th = snap[j]["theta"].copy()
        pays = []
        for r in range(3):
            if r == 1:
                pays.append(None)
                continue
            out = O.compress(cfg, tab, snap[j]["theta"], snap[j]["local"][r], snap[j]["e"][r].copy())
            assert np.array_equal(c.tensor_payload(r, j), out.payload), (t.name, r)
            pays.append(out.payload)
        O.aggregate_apply(cfg, tab, pays, th)
        got = c.theta[c.offs[j]:c.offs[j] + t.numel].cpu().numpy()
        rms = float(np.sqrt(np.mean(th.astype(np.float64) ** 2)))
        assert float(np.max(np.abs(got.astype(np.float64) - th.astype(np.float64)))) <= 1e-6 * rms
    from paper_2508_15706_b200 import binding as B
    with pytest.raises(B.SlError) as ei:     # the wire codec and deferral serve the 2-bit payload only
        c.sl.coded_payload_capacity()
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError):
        c.sl.set_ef_deferred(True)


@pytest.mark.parametrize("bits,k", [(2, 257), (2, 512), (2, 2048), (4, 1000), (1, 2048)])
def test_densities_up_to_half_a_chunk(bits, k):
    """k beyond 256, up to 2048 of 4096 (the densest setting of the paper's density sweeps): the whole
    outer step against the oracle, payload and error buffers bit for bit, theta within 1e-6 x RMS, two
    steps; chunks shorter than k send all they have."""
    from parity import DeviceCase, oracle_threads
    oracle_threads()
    tensors = TENSORS + [I.TensorSpec("big", 576, 512, 5)]
    wl = I.Workload("dense_k", tensors, R=3, k=k, recipe="student_t4", seed=400 + k + bits, outer_lr=0.7)
    c = DeviceCase(wl, e_scale=0.5, quant_bits=bits)
    assert c.sl.payload_bytes() == c.payload_bytes
    for step in range(2):
        c.fill_local(step)
        snap = c.snapshot(range(len(tensors)))
        c.step()
        rep = c.check(snap)
        assert rep["tensors"] == len(tensors)
    from paper_2508_15706_b200 import binding as B
    with pytest.raises(B.SlError) as ei:     # deferral and the wire codec stop at k = 256
        c.sl.set_ef_deferred(True)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:     # and so does the path without a quantiser
        B.SparseLoCo(c.shapes, c.offs, k=k, R=3, quant_bits=32, alloc_workspace=False)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo(c.shapes, c.offs, k=2049, R=3, alloc_workspace=False)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
