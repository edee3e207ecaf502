"""Pins for the oracle's quantiser at 1, 3 and 4 bits (Sec. 4; the paper's ablation over quantisation
widths) and for the payload format that carries such codes: hand-worked cases (tests/golden), the 2-bit
routine reproduced bit for bit by the general one, an independent floor-based restatement of the binning,
invariants (monotone codes, centroids, empty bins), pack/unpack round trips and the closed-form sizes."""
import math
import os

import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLD, "handworked_quantiser_widths.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = {"name": tok[1]}
            cases.append(cur)
        else:
            cur[tok[0]] = [float(x) for x in tok[1:]]
    return cases


@pytest.mark.parametrize("case", read_cases(), ids=lambda c: c["name"])
def test_handworked(case):
    v = np.array(case["v"], np.float32)
    bits = int(case["bits"][0])
    for split in ([v.size], [3, v.size - 3]):
        mu, sigma, lut, code = O.quantize_tensor_q(v, np.array(split, np.int32), bits)
        assert mu == np.float32(case["mu"][0])
        assert abs(float(sigma) - case["sigma"][0]) < 1e-5
        assert list(code) == [int(c) for c in case["codes"]]
        assert np.allclose(lut, np.array(case["lut"], np.float32), rtol=1e-6, atol=0)


@pytest.mark.parametrize("n_chunks", [1, 7, 65, 300])
def test_two_bits_is_the_special_routine(n_chunks):
    rng = np.random.default_rng(70 + n_chunks)
    cnt = rng.integers(1, 65, n_chunks).astype(np.int32)
    v = (rng.standard_t(3, int(cnt.sum())) * 1e-3 + 2e-4).astype(np.float32)
    a = O.quantize_tensor(v, cnt)
    b = O.quantize_tensor_q(v, cnt, 2)
    assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32)) and np.array_equal(a[3], b[3])


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_binning_against_a_floor_restatement_and_invariants(bits):
    rng = np.random.default_rng(80 + bits)
    nb = 1 << bits
    cnt = np.full(40, 64, np.int32)
    v = (rng.standard_normal(40 * 64) * 2e-3 + 5e-4).astype(np.float32)
    v[:5] = [0.1, -0.1, 0.05, -0.02, 0.011]        # beyond 6 sigma: outer bins
    mu, sigma, lut, code = O.quantize_tensor_q(v, cnt, bits)
    v64 = v.astype(np.float64)
    assert abs(float(mu) - v64.mean()) <= 2 ** -23 * abs(v64.mean())
    cen = (v - mu).astype(np.float32).astype(np.float64)
    assert abs(float(sigma) - math.sqrt((cen ** 2).mean())) <= 2 ** -23 * float(sigma)
    # uniform bins of width 12 sigma / 2^bits over [-6 sigma, 6 sigma], outer bins open-ended
    width = 12.0 * float(sigma) / nb
    want = np.clip(np.floor((cen + 6.0 * float(sigma)) / width), 0, nb - 1).astype(int)
    near_edge = np.abs((cen + 6.0 * float(sigma)) / width - np.round((cen + 6.0 * float(sigma)) / width)) < 1e-4
    assert np.array_equal(code[~near_edge], want[~near_edge])
    assert code[0] == nb - 1 and code[1] == 0
    order = np.argsort(v, kind="stable")
    assert np.all(np.diff(code[order].astype(int)) >= 0)                       # codes monotone in the value
    for b in range(nb):
        m = code == b
        if m.any():
            assert abs(float(lut[b]) - v64[m].mean()) <= 2 ** -22 * abs(v64[m].mean()) + 1e-45
        else:
            assert lut[b] == 0.0
    dec = lut[code].astype(np.float64)
    assert abs(dec.sum() - v64.sum()) <= 1e-6 * np.abs(v64).sum()               # centroids preserve the sum


def test_more_bits_leave_a_smaller_residual():
    rng = np.random.default_rng(90)
    v = rng.standard_normal(64 * 50).astype(np.float32)
    cnt = np.full(50, 64, np.int32)
    res = []
    for bits in (1, 2, 3, 4):
        _, _, lut, code = O.quantize_tensor_q(v, cnt, bits)
        res.append(float(np.sum((v - lut[code]) ** 2)))
    assert res[0] > res[1] > res[2] > res[3]


@pytest.mark.parametrize("bits,k", [(1, 64), (3, 41), (4, 64), (3, 123), (4, 5)])
def test_record_round_trip_and_sizes(bits, k):
    rng = np.random.default_rng(100 + bits + k)
    idx = np.sort(rng.choice(4096, size=k, replace=False)).astype(np.int32)
    code = rng.integers(0, 1 << bits, k).astype(np.uint8)
    rec = O.pack_record_q(idx, code, k, bits)
    assert rec.size == O.record_stride_q(k, bits) == ((12 * k + 7) // 8 + (bits * k + 7) // 8 + 15) // 16 * 16
    i2, c2 = O.unpack_record_q(rec, k, k, bits)
    assert np.array_equal(i2, idx) and np.array_equal(c2, code)
    # index block as at 2 bits; the code block starts at the same byte
    assert np.array_equal(rec[:(12 * k + 7) // 8], O.pack_record(idx, np.zeros(k, np.uint8), k)[:(12 * k + 7) // 8])
    assert O.header_bytes(bits) == max(16, 4 << bits)
    if bits == 2:
        assert O.record_stride_q(k, 2) == O.record_stride(k)


@pytest.mark.parametrize("bits", [1, 3, 4])
def test_compress_decode_round_trip(bits):
    rng = np.random.default_rng(110 + bits)
    shapes = [(128, 64), (1, 5000)]
    tab = O.Table(shapes)
    cfg = O.Config(k=41, R=2, quant_bits=bits)
    n = tab.numel
    theta = rng.standard_normal(n).astype(np.float32)
    local = (theta - 0.01 * rng.standard_normal(n)).astype(np.float32)
    e = (0.005 * rng.standard_normal(n)).astype(np.float32)
    u = O.ef_accumulate(theta, local, e, cfg.beta)
    out = O.compress(cfg, tab, theta, local, e)
    assert out.payload.size == O.payload_bytes(cfg, tab) == 2 * O.header_bytes(bits) + O.record_stride_q(41, bits) * O.total_chunks(cfg, tab)
    idx, hat = O.decode_payload(cfg, tab, out.payload)
    assert np.array_equal(idx, out.sel_idx) and np.array_equal(hat.view(np.uint32), out.sel_hat.view(np.uint32))
    # error feedback identity (Eq. 2): what was sent plus what stays behind is u
    sent = np.zeros(n, np.float64)
    w = 0
    for j, (r, c) in enumerate(shapes):
        for ch in range(O.num_chunks(cfg, tab, j)):
            L = O.chunk_len(cfg, tab, j, ch)
            for s in range(min(41, L)):
                sent[tab.shapes[j][2] + O.chunk_pos(cfg, tab, j, ch, int(out.sel_idx[w]))] = out.sel_hat[w]
                w += 1
    assert np.allclose(e.astype(np.float64) + sent, u.astype(np.float64), rtol=0, atol=1e-7)
    # and two workers' payloads aggregate as at 2 bits
    th = theta.copy()
    O.aggregate_apply(cfg, tab, [out.payload, out.payload], th)
    assert np.allclose(th.astype(np.float64), theta.astype(np.float64) - cfg.outer_lr * sent, rtol=0, atol=1e-6)
