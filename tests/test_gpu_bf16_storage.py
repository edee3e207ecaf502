"""bfloat16 storage of theta, theta_local and e (sl_*_bf16) against the oracle's storage mode.
The paper names no storage type; the definition both sides follow: the fp32 arithmetic of the method on
the widened values, selection and quantiser on the unrounded u, one round-to-nearest-even per store.
Bars: payload bytes and error buffers bit for bit.  theta: the kernel rounds fma(-alpha/D, fp32 sum,
theta), the oracle rounds the fp64 expression; the two fp32/fp64 values differ by about 1e-7 of the
update, so they land on different sides of a rounding boundary for about one element in a million:
every element must be within one bfloat16 step and at most 1e-4 of them may differ at all."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu

TENSORS = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 5000, 0), I.TensorSpec("router", 8, 1024, 1),
           I.TensorSpec("norm", 1, 768, 1), I.TensorSpec("tiny", 1, 40, 2), I.TensorSpec("big", 576, 512, 3)]
PAD = 2048  # elements of a known pattern after every array: must come back untouched


def _padded(t: torch.Tensor) -> torch.Tensor:
    out = torch.full((t.numel() + PAD,), 1.5, dtype=torch.bfloat16, device=t.device)
    out[:t.numel()] = t.to(torch.bfloat16)
    return out


def _widen(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float32).cpu().numpy()


@pytest.mark.parametrize("bits,k,R,deferred", [(2, 64, 3, False), (2, 64, 3, True), (2, 41, 2, False), (2, 200, 5, True),
                                               (2, 1, 1, True), (4, 64, 2, False), (1, 200, 2, False), (2, 600, 2, False),
                                               (3, 300, 1, False)])
def test_outer_step_bf16_against_oracle(bits, k, R, deferred):
    from paper_2508_15706_b200 import binding as B
    O.set_threads(8)
    dev = torch.device("cuda", torch.cuda.current_device())
    wl = I.Workload("bf16", TENSORS, R=R, k=k, recipe="student_t4", seed=900 + k + bits, outer_lr=0.7, beta=0.9)
    shapes, offs = [(t.rows, t.cols) for t in TENSORS], I.offsets(TENSORS)
    n = offs[-1] + TENSORS[-1].numel
    sl = B.SparseLoCo(shapes, offs, k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=bits, bf16_storage=True)
    cfg = O.Config(k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, quant_bits=bits, storage_bf16=1)
    tab = O.Table(shapes, offs)
    assert sl.payload_bytes() == O.payload_bytes(cfg, tab)
    if deferred:   # the corrected values wait (as fp32) in the workspace and are rounded when they reach e
        sl.set_ef_deferred(True)
    theta = _padded(I.theta_sync(wl, dev))
    e = [_padded(I.initial_error(wl, r, dev, scale=0.5)) for r in range(R)]
    pay = [torch.full((sl.payload_bytes() + 64,), 0xC5, dtype=torch.uint8, device=dev) for _ in range(R)]
    th_o = _widen(theta[:n])
    e_o = [_widen(x[:n]) for x in e]
    for step in range(3):
        local = [_padded(I.theta_local(wl, theta[:n].to(torch.float32), r, step)) for r in range(R)]
        lo_o = [_widen(x[:n]) for x in local]
        sl.outer_step(theta, local, e, pay)
        torch.cuda.synchronize()
        assert sl.device_status() == 0
        want = O.outer_step(cfg, tab, th_o, lo_o, e_o)
        true_e = e
        if deferred:   # the error as the method defines it: the waiting values written into copies
            assert sl.ef_pending()
            true_e = [x.clone() for x in e]
            sl.ef_flush(true_e, keep_pending=True)
            torch.cuda.synchronize()
        for r in range(R):
            assert np.array_equal(pay[r][:-64].cpu().numpy(), want[r]), f"payload of worker {r}, step {step}"
            assert bool((pay[r][-64:] == 0xC5).all())
            got_e = _widen(true_e[r][:n])
            assert np.array_equal(got_e.view(np.uint32), e_o[r].view(np.uint32)), f"e of worker {r}, step {step}"
            assert bool((e[r][n:] == 1.5).all()) and bool((local[r][n:] == 1.5).all())
        got = _widen(theta[:n])
        assert bool((theta[n:] == 1.5).all())
        diff = np.nonzero(got != th_o)[0]
        assert diff.size <= max(1, int(1e-4 * n)), (diff.size, n)
        for i in diff:  # neighbours on the bfloat16 grid
            a, b = int(got.view(np.uint32)[i]) >> 16, int(th_o.view(np.uint32)[i]) >> 16
            assert abs(a - b) == 1, (i, got[i], th_o[i])
        th_o = got.copy()  # both sides continue from the same parameters
    if deferred:
        sl.ef_flush()
        torch.cuda.synchronize()
        assert not sl.ef_pending()
        for r in range(R):
            assert np.array_equal(_widen(e[r][:n]).view(np.uint32), e_o[r].view(np.uint32))
            assert bool((e[r][n:] == 1.5).all())


def test_halves_through_their_own_entry_points_and_type_checks():
    """sl_compress_bf16 / sl_aggregate_apply_bf16 with an absent worker; the fp32 calls refuse a bfloat16
    context and the other way round."""
    import ctypes as C
    from paper_2508_15706_b200 import binding as B
    O.set_threads(8)
    dev = torch.device("cuda", torch.cuda.current_device())
    R, k = 3, 64
    wl = I.Workload("bf16h", TENSORS, R=R, k=k, recipe="student_t4", seed=77, outer_lr=0.9, beta=0.9)
    shapes, offs = [(t.rows, t.cols) for t in TENSORS], I.offsets(TENSORS)
    n = offs[-1] + TENSORS[-1].numel
    sl = B.SparseLoCo(shapes, offs, k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, bf16_storage=True,
                      divide_by_present=True)
    cfg = O.Config(k=k, R=R, beta=wl.beta, outer_lr=wl.outer_lr, storage_bf16=1, divide_by_present=1)
    tab = O.Table(shapes, offs)
    theta = I.theta_sync(wl, dev).to(torch.bfloat16)
    th_o = _widen(theta)
    pays, want = [], []
    for r in range(R):
        if r == 1:
            pays.append(None)
            want.append(None)
            continue
        local = I.theta_local(wl, theta.to(torch.float32), r, 0).to(torch.bfloat16)
        e = I.initial_error(wl, r, dev, scale=0.5).to(torch.bfloat16)
        e_o = _widen(e)
        p = torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev)
        sl.compress(theta, local, e, p)
        out = O.compress(cfg, tab, th_o, _widen(local), e_o)
        torch.cuda.synchronize()
        assert np.array_equal(p.cpu().numpy(), out.payload)
        assert np.array_equal(_widen(e).view(np.uint32), e_o.view(np.uint32))
        pays.append(p)
        want.append(out.payload)
    sl.aggregate_apply(pays, theta)
    O.aggregate_apply(cfg, tab, want, th_o)
    torch.cuda.synchronize()
    got = _widen(theta)
    diff = np.nonzero(got != th_o)[0]
    assert diff.size <= max(1, int(1e-4 * n))
    for i in diff:
        assert abs((int(got.view(np.uint32)[i]) >> 16) - (int(th_o.view(np.uint32)[i]) >> 16)) == 1
    # element types are fixed by the context
    f32 = torch.zeros(n, device=dev)
    p = torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev)
    st = B._L.sl_compress(sl._h, f32.data_ptr(), f32.data_ptr(), f32.data_ptr(), p.data_ptr(), None)
    assert st == B.SL_ERR_UNSUPPORTED
    sl32 = B.SparseLoCo(shapes, offs, k=k, R=R)
    st = B._L.sl_compress_bf16(sl32._h, theta.data_ptr(), theta.data_ptr(), theta.data_ptr(), p.data_ptr(), None)
    assert st == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:
        B.SparseLoCo(shapes, offs, k=k, R=R, bf16_storage=True, quant_bits=32)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    with pytest.raises(B.SlError) as ei:     # the fused update from coded payloads works on fp32 arrays
        sl.aggregate_apply_coded([p, None, None], theta)
    assert ei.value.status == B.SL_ERR_UNSUPPORTED
    # the wire codec and the validator are about payloads, not about storage
    cap = sl.coded_payload_capacity()
    coded = torch.zeros(cap, dtype=torch.uint8, device=dev)
    size = torch.zeros(1, dtype=torch.int64, device=dev)
    sl.encode_payload(pays[0], coded, size)
    back = torch.zeros_like(pays[0])
    sl.decode_payload(coded, back, int(size.item()))
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    sl.validate_payload(back, status)
    torch.cuda.synchronize()
    assert torch.equal(back, pays[0]) and status.item() == 0
