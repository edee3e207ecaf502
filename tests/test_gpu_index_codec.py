"""GPU parity of the entropy-coded index format: sl_encode_payload must produce exactly the oracle's
coded bytes (and size) from the payloads the compression wrote, sl_decode_payload must restore the
12-bit payload bit for bit, at small sizes with every chunk shape and at the 2B config's full size."""
import gc

import numpy as np
import pytest
import torch

import oracle as O
from paper_2508_15706_b200 import inputs as I

pytestmark = pytest.mark.gpu

SHAPES = [I.TensorSpec("a", 128, 192, 0), I.TensorSpec("flat", 1, 5000, 0), I.TensorSpec("tiny", 1, 40, 1),
          I.TensorSpec("norm", 1, 768, 1), I.TensorSpec("long", 1, 4096 * 40 + 3, 2), I.TensorSpec("b", 64, 64, 2)]


def _case(wl, **kw):
    from parity import DeviceCase, oracle_threads
    gc.collect()
    torch.cuda.empty_cache()
    oracle_threads()
    return DeviceCase(wl, **kw)


@pytest.mark.parametrize("k", [1, 8, 41, 64, 123, 256])
def test_encode_matches_oracle_and_decode_restores(k):
    wl = I.Workload("codec", SHAPES, R=2, k=k, recipe="student_t4", seed=700 + k)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    c.step()
    cap = c.sl.coded_payload_capacity()
    tab = O.Table(c.shapes, c.offs)
    cfg = O.Config(k=k, R=2)
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    for r in range(2):
        coded = torch.full((cap,), 0x5A, dtype=torch.uint8, device=c.dev)  # stale bytes must not leak into the result
        c.sl.encode_payload(c.payloads[r], coded, size)
        torch.cuda.synchronize()
        want = O.ixc_encode_payload(cfg, tab, c.payloads[r].cpu().numpy())
        n = int(size.item())
        assert n == want.size and n <= cap
        assert np.array_equal(coded[:n].cpu().numpy(), want)
        back = torch.full_like(c.payloads[r], 0xA5)
        c.sl.decode_payload(coded, back)
        torch.cuda.synchronize()
        assert torch.equal(back, c.payloads[r])


def test_full_size_round_trip_and_rate():
    """The 2B config, one worker's payload: round trip on the GPU, size equal to the oracle's, and the
    index rate it reaches on these (non-uniform) index sets."""
    wl = I.workload("c5_dense_d2048")
    import dataclasses
    wl = dataclasses.replace(wl, R=1)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    c.step()
    cap = c.sl.coded_payload_capacity()
    coded = torch.empty(cap, dtype=torch.uint8, device=c.dev)
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    c.sl.encode_payload(c.payloads[0], coded, size)
    back = torch.empty_like(c.payloads[0])
    c.sl.decode_payload(coded, back)
    torch.cuda.synchronize()
    assert torch.equal(back, c.payloads[0])
    n = int(size.item())
    want = O.ixc_encode_payload(O.Config(k=wl.k), O.Table(c.shapes, c.offs), c.payloads[0].cpu().numpy())
    assert n == want.size
    assert np.array_equal(coded[:n].cpu().numpy(), want)
    chunks, slots = c.sl.num_chunks()
    T = len(c.shapes)
    index_bits = 8 * (n - 16 * T - 16 * chunks) / slots   # code blocks are 16 bytes per chunk at k = 64
    assert index_bits < 8.0, index_bits                   # 12 in the plain format; 7.36 is the bound at k = 64
    assert n < 0.72 * c.sl.payload_bytes()


def test_damaged_coded_payloads_stay_inside_the_buffer():
    """A coded payload damaged on the host -- directory entries far beyond the stream, a directory
    that goes backwards, a stream of all ones, a truncated buffer -- is decoded without reading past
    the bytes the caller declared (the decoder clamps every position to them) and the damage is
    reported: SL_ERR_BAD_PAYLOAD in the status word and / or a record sl_validate_payload rejects.
    The coded buffer is a slice that ends exactly at the declared size, inside a larger allocation
    filled with a canary, so the bytes behind it are known and the output must not depend on them."""
    wl = I.Workload("ixc_bad", [I.TensorSpec("w", 512, 512, 0), I.TensorSpec("v", 1, 5000, 0)], R=1, k=64,
                    recipe="normal", seed=5)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    c.step()
    cap = c.sl.coded_payload_capacity()
    good = torch.zeros(cap, dtype=torch.uint8, device=c.dev)
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    c.sl.encode_payload(c.payloads[0], good, size)
    torch.cuda.synchronize()
    n = int(size.item())
    chunks, _ = c.sl.num_chunks()
    T = len(c.shapes)
    dir_off = (16 * T + 16 * chunks + 3) // 4 * 4
    n_dir = (chunks + 15) // 16
    stream_off = dir_off + 4 * n_dir
    status = torch.zeros(1, dtype=torch.int32, device=c.dev)

    def run(mutate, declared):
        host = good[:n].cpu().numpy().copy()
        mutate(host)
        arena = torch.full((cap + 4096,), 0xEE, dtype=torch.uint8, device=c.dev)
        arena[:declared] = torch.from_numpy(host[:declared]).to(c.dev)
        outs = []
        for canary in (0xEE, 0x11):  # whatever lies behind the declared bytes must not matter
            arena[declared:] = canary
            back = torch.full_like(c.payloads[0], 0xA5)
            c.sl.decode_payload(arena, back, coded_bytes=declared)
            dev_status = c.sl.device_status()
            c.sl.validate_payload(back, status)
            torch.cuda.synchronize()
            outs.append((back.cpu().numpy().copy(), dev_status, int(status.item())))
        assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1:] == outs[1][1:]
        return outs[0]

    # untouched: round trip, nothing reported
    back, st, val = run(lambda h: None, n)
    assert st == 0 and val == 0 and np.array_equal(back, c.payloads[0].cpu().numpy())

    def far_directory(h):
        h[dir_off + 4:dir_off + 8] = np.frombuffer(np.uint32(0xFFFFFF00).tobytes(), np.uint8)
    back, st, val = run(far_directory, n)
    assert st == 4

    def backwards_directory(h):
        h[dir_off + 8:dir_off + 12] = 0
    back, st, val = run(backwards_directory, n)
    assert st == 4

    def all_ones(h):
        h[stream_off:] = 0xFF
    back, st, val = run(all_ones, n)
    assert st == 4 or val == 4

    back, st, val = run(lambda h: None, stream_off + 16)  # truncated: most of the stream is missing
    assert st == 4


@pytest.mark.parametrize("k,R", [(1, 2), (8, 3), (41, 3), (64, 16), (123, 5), (256, 3), (64, 40), (200, 64), (1, 1)])
def test_aggregate_apply_straight_from_coded_payloads(k, R):
    """sl_aggregate_apply_coded (the decoding fused into the update kernel; Eq. 2 lines 3-4) must leave the
    bits that sl_decode_payload for every worker + sl_aggregate_apply leave, with an absent worker and with
    the exact coded sizes as read limits; and agree with the oracle's update within 1e-6 x RMS."""
    wl = I.Workload("codec_apply", SHAPES, R=R, k=k, recipe="student_t4", seed=800 + k + R, outer_lr=0.7)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    c.step()
    cap = c.sl.coded_payload_capacity()
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    coded, sizes = [], []
    for r in range(R):
        buf = torch.full((cap,), 0x5A, dtype=torch.uint8, device=c.dev)
        c.sl.encode_payload(c.payloads[r], buf, size)
        sizes.append(int(size.item()))
        coded.append(buf)
    absent = 1 if R > 1 else None
    plain = [None if r == absent else c.payloads[r] for r in range(R)]
    theta_a = c.theta.clone()
    c.sl.aggregate_apply(plain, theta_a)
    theta_b = torch.cat([c.theta.clone(), torch.full((1024,), 7.5, device=c.dev)])  # a band that must survive
    c.sl.aggregate_apply_coded([None if r == absent else coded[r] for r in range(R)], theta_b, sizes)
    torch.cuda.synchronize()
    assert c.sl.device_status() == 0
    n = c.theta.numel()
    assert torch.equal(theta_b[:n].view(torch.int32), theta_a.view(torch.int32))
    assert bool((theta_b[n:] == 7.5).all())
    # the oracle on the same payloads
    tab = O.Table(c.shapes, c.offs)
    cfg = O.Config(k=k, R=R, outer_lr=wl.outer_lr)
    th = c.theta.cpu().numpy().copy()
    O.aggregate_apply(cfg, tab, [None if p is None else p.cpu().numpy() for p in plain], th)
    rms = float(np.sqrt(np.mean(th.astype(np.float64) ** 2)))
    assert float(np.max(np.abs(theta_b[:n].cpu().numpy().astype(np.float64) - th))) <= 1e-6 * rms


def test_coded_apply_with_a_cut_stream_stays_in_bounds_and_reports():
    """A coded payload whose stated size cuts the index stream short: the update of that call is wrong by
    definition, but every access stays inside the stated sizes and inside theta, and the device status
    says SL_ERR_BAD_PAYLOAD."""
    from paper_2508_15706_b200 import binding as B
    k, R = 64, 2
    wl = I.Workload("codec_cut", SHAPES, R=R, k=k, recipe="student_t4", seed=31, outer_lr=0.7)
    c = _case(wl, e_scale=0.5)
    c.fill_local(0)
    c.step()
    cap = c.sl.coded_payload_capacity()
    size = torch.zeros(1, dtype=torch.int64, device=c.dev)
    coded, sizes = [], []
    for r in range(R):
        buf = torch.zeros(cap, dtype=torch.uint8, device=c.dev)
        c.sl.encode_payload(c.payloads[r], buf, size)
        sizes.append(int(size.item()))
        coded.append(buf)
    # the buffer really ends where the call is told it ends: a copy of exactly that many bytes
    cut = (sizes[0] + c.sl.coded_payload_capacity() * 0) // 2 // 16 * 16
    fixed = 16 * len(c.shapes)  # (tables; the stream starts well after this)
    assert cut > fixed
    short = coded[0][:cut].clone()
    theta = torch.cat([c.theta.clone(), torch.full((1024,), 7.5, device=c.dev)])
    try:
        c.sl.aggregate_apply_coded([short, coded[1]], theta, [cut, sizes[1]])
        torch.cuda.synchronize()
        st = c.sl.device_status()
        assert st == B.SL_ERR_BAD_PAYLOAD
    except B.SlError as e:   # a size that does not even reach the stream is refused on the host
        assert e.status == B.SL_ERR_INVALID_ARG
    assert bool((theta[c.theta.numel():] == 7.5).all())
    assert bool(torch.isfinite(theta).all())
