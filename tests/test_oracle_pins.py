"""Pins for the CPU oracle: each test checks it against something other than itself --
brute force written independently here, exact rational arithmetic, hand-worked cases
(tests/golden), closed forms and values the paper prints, invariants, and special cases that
reduce to a library routine (numpy mean / reshape)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers

def read_kv(path):
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def f32_round_exact(x: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) fp32 of an exact rational."""
    if x == 0:
        return np.float32(0.0)
    g = np.float32(float(x))  # close guess; refine among neighbours using exact distances
    cands = {g, np.nextafter(g, np.float32(np.inf)), np.nextafter(g, np.float32(-np.inf))}
    best = None
    for c in cands:
        if not np.isfinite(c):
            continue
        d = abs(Fraction(float(c)) - x)
        even = (np.array([c]).view(np.uint32)[0] & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def brute_topk(u: np.ndarray, k: int) -> np.ndarray:
    """k rounds of 'largest remaining magnitude, lowest index on ties'.  Independent of sorting."""
    key = (u.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)
    alive = np.ones(u.size, bool)
    out = []
    for _ in range(min(k, u.size)):
        best, bi = -1, -1
        for i in range(u.size):
            if alive[i] and key[i] > best:
                best, bi = key[i], i
        alive[bi] = False
        out.append(bi)
    return np.array(sorted(out), np.int32)


# ----------------------------------------------------------------------------- error feedback

def test_ef_accumulate_is_single_rounded_fma():
    rng = np.random.default_rng(1)
    n = 300
    theta = rng.standard_normal(n).astype(np.float32)
    theta_r = (theta + rng.standard_normal(n).astype(np.float32) * np.float32(1e-3)).astype(np.float32)
    e = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    # a few adversarial rows: product lands next to a rounding boundary of the sum
    theta[:3] = [1.0, 0.0, 3.0]
    theta_r[:3] = [0.0, -1.0, 1.0]
    e[:3] = [np.float32(2.0 ** -24) * np.float32(1 / 0.95), np.float32(2.0 ** -25), np.float32(2.0 ** -23 + 2.0 ** -46)]
    beta = np.float32(0.95)
    u = O.ef_accumulate(theta, theta_r, e, float(beta))
    for i in range(n):
        d = np.float32(theta[i] - theta_r[i])  # fp32 subtraction
        exact = Fraction(float(beta)) * Fraction(float(e[i])) + Fraction(float(d))
        want = f32_round_exact(exact)
        assert u[i].tobytes() == want.tobytes(), (i, u[i], want)


def test_ef_accumulate_freeze_and_beta_zero():
    rng = np.random.default_rng(2)
    theta = rng.standard_normal(64).astype(np.float32)
    theta_r = rng.standard_normal(64).astype(np.float32)
    e = rng.standard_normal(64).astype(np.float32)
    d = theta - theta_r
    assert np.array_equal(O.ef_accumulate(theta, theta_r, e, 0.95, ef_enabled=0), d)
    assert np.array_equal(O.ef_accumulate(theta, theta_r, e, 0.0), d)
    # beta = 1, theta == theta_r: u = e
    assert np.array_equal(O.ef_accumulate(theta, theta, e, 1.0), e)


# ----------------------------------------------------------------------------- Top-k

@pytest.mark.parametrize("L,k", [(16, 1), (16, 5), (16, 16), (16, 20), (64, 7), (64, 63), (100, 33), (1, 1),
                                 (4096, 257), (4096, 512), (4096, 2048), (4096, 4095), (4096, 4096), (3000, 2048)])
def test_topk_matches_bruteforce(L, k):
    """(the densities of the paper's sweeps go up to 50 %, k = 2048 of 4096)"""
    rng = np.random.default_rng(L * 100 + k)
    for trial in range(20 if L <= 100 else 3):
        u = rng.standard_normal(L).astype(np.float32)
        if trial % 3 == 1:  # heavy ties, both signs
            u = (rng.integers(-2, 3, L)).astype(np.float32)
        if trial % 3 == 2:  # few distinct magnitudes with zeros and denormals
            u = rng.choice(np.array([0.0, -0.0, 1e-42, -1e-42, 2.5, -2.5, 7.0], np.float32), L)
        got = O.topk_chunk(u, k)
        want = brute_topk(u, k)
        assert np.array_equal(got, want), (trial, u, got, want)


def test_topk_invariants_full_chunk():
    rng = np.random.default_rng(7)
    for k in (1, 41, 64, 123, 256, 300, 1024, 2048):
        u = rng.standard_normal(4096).astype(np.float32)
        u[rng.integers(0, 4096, 300)] = np.float32(0.5)  # a tie group
        idx = O.topk_chunk(u, k)
        assert idx.size == k and np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < 4096
        key = u.view(np.uint32) & np.uint32(0x7FFFFFFF)
        sel = np.zeros(4096, bool)
        sel[idx] = True
        kmin = key[sel].min()
        assert kmin >= key[~sel].max()
        tied_sel = np.nonzero(sel & (key == kmin))[0]
        tied_uns = np.nonzero(~sel & (key == kmin))[0]
        if tied_uns.size:
            assert tied_sel.max() < tied_uns.min()


def test_topk_degenerate_inputs():
    z = np.zeros(4096, np.float32)
    assert np.array_equal(O.topk_chunk(z, 64), np.arange(64, dtype=np.int32))
    z[1::2] = -0.0  # -0 ties with +0
    assert np.array_equal(O.topk_chunk(z, 64), np.arange(64, dtype=np.int32))
    u = np.array([1.0, -np.inf, np.nan, 3.0, 1e-45, -1e-45, 0.0], np.float32)
    # NaN (largest bit pattern) > Inf > 3 > 1 > denormals (tie, lower index first) > 0
    assert list(O.topk_chunk(u, 1)) == [2]
    assert list(O.topk_chunk(u, 2)) == [1, 2]
    assert list(O.topk_chunk(u, 5)) == [0, 1, 2, 3, 4]
    assert list(O.topk_chunk(u, 6)) == [0, 1, 2, 3, 4, 5]
    assert list(O.topk_chunk(u, 99)) == [0, 1, 2, 3, 4, 5, 6]
    # sign does not matter
    v = np.array([0.1, -0.9, 0.5, -0.2], np.float32)
    assert list(O.topk_chunk(v, 2)) == [1, 2]


# ----------------------------------------------------------------------------- chunk geometry

def test_tile_geometry_matches_numpy_reshape():
    cfg = O.Config(k=2, chunk_elems=4, tile_dim=2)
    rows, cols = 4, 6
    tab = O.Table([(rows, cols)])
    A = np.arange(rows * cols).reshape(rows, cols)
    want = A.reshape(rows // 2, 2, cols // 2, 2).transpose(0, 2, 1, 3).reshape(-1, 4)
    assert O.num_chunks(cfg, tab, 0) == want.shape[0] == 6
    for ch in range(6):
        assert O.chunk_len(cfg, tab, 0, ch) == 4
        got = [O.chunk_pos(cfg, tab, 0, ch, p) for p in range(4)]
        assert got == list(want[ch]), (ch, got)
    # hand-written: chunk 1 of a 4x6 matrix in 2x2 blocks = rows 0-1, cols 2-3
    assert [O.chunk_pos(cfg, tab, 0, 1, p) for p in range(4)] == [2, 3, 8, 9]
    assert [O.chunk_pos(cfg, tab, 0, 3, p) for p in range(4)] == [12, 13, 18, 19]


def test_flat_geometry_and_fallbacks():
    cfg = O.Config(k=64)
    tab = O.Table([(1, 10000), (8, 1024), (70, 64), (128, 192)])
    assert O.num_chunks(cfg, tab, 0) == 3
    assert [O.chunk_len(cfg, tab, 0, c) for c in range(3)] == [4096, 4096, 10000 - 8192]
    assert O.chunk_pos(cfg, tab, 0, 2, 5) == 8197
    # 8 x 1024: rows not a multiple of 64 -> flat runs
    assert O.num_chunks(cfg, tab, 1) == 2 and O.chunk_pos(cfg, tab, 1, 1, 0) == 4096
    # 70 x 64 -> flat, 4480 elements -> 2 chunks, tail of 384
    assert O.num_chunks(cfg, tab, 2) == 2 and O.chunk_len(cfg, tab, 2, 1) == 384
    # 128 x 192 -> 2 x 3 blocks; block 4 = block-row 1, block-col 1; p = 65 -> row 64+1, col 64+1
    assert O.num_chunks(cfg, tab, 3) == 6
    assert O.chunk_pos(cfg, tab, 3, 4, 65) == (64 + 1) * 192 + 64 + 1
    assert O.total_chunks(cfg, tab) == 3 + 2 + 2 + 6
    assert O.total_slots(cfg, tab) == 64 * 13
    cfg2 = O.Config(k=100)
    tab2 = O.Table([(1, 4096 + 70)])
    assert O.total_slots(cfg2, tab2) == 100 + 70


# ----------------------------------------------------------------------------- quantiser

def read_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLD, "handworked_quantiser.txt")):
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
def test_quantiser_handworked(case):
    v = np.array(case["v"], np.float32)
    for split in ([v.size], [1, v.size - 1] if v.size > 1 else [1], [v.size // 2, v.size - v.size // 2]):
        mu, sigma, lut, code = O.quantize_tensor(v, np.array(split, np.int32))
        assert mu == np.float32(case["mu"][0])
        assert abs(float(sigma) - case["sigma"][0]) < 1e-4
        assert list(code) == [int(c) for c in case["codes"]]
        assert list(lut) == [np.float32(x) for x in case["lut"]]


def test_quantiser_invariants_random():
    rng = np.random.default_rng(5)
    for n_chunks, k in ((1, 64), (7, 64), (40, 41), (3, 123)):
        v = (rng.standard_t(3, n_chunks * k) * 1e-3 + 2e-4).astype(np.float32)
        cnt = np.full(n_chunks, k, np.int32)
        mu, sigma, lut, code = O.quantize_tensor(v, cnt)
        v64 = v.astype(np.float64)
        # mean and population sigma against numpy (fp64), to fp32 rounding
        assert abs(float(mu) - v64.mean()) <= 2 ** -24 * abs(v64.mean()) * 1.01 + 1e-45
        cen = (v - mu).astype(np.float32).astype(np.float64)
        assert abs(float(sigma) - math.sqrt((cen ** 2).mean())) <= 2 ** -23 * float(sigma)
        t = np.float32(3.0) * sigma
        # codes monotone in v and consistent with the edges
        order = np.argsort(v, kind="stable")
        assert np.all(np.diff(code[order].astype(int)) >= 0)
        c32 = (v - mu).astype(np.float32)
        assert np.all((code == 0) == (c32 < -t)) and np.all((code == 3) == (c32 >= t))
        assert np.all((code >= 2) == (c32 >= 0))
        # centroids: per bin the mean of the raw values; residuals sum to ~0; decoded sum = raw sum
        for b in range(4):
            m = code == b
            if m.any():
                assert abs(float(lut[b]) - v64[m].mean()) <= 2 ** -23 * abs(v64[m].mean()) + 1e-45
            else:
                assert lut[b] == 0.0
        nonempty = [float(lut[b]) for b in range(4) if (code == b).any()]
        assert nonempty == sorted(nonempty)
        dec = lut[code].astype(np.float64)
        assert abs(dec.sum() - v64.sum()) <= 1e-6 * np.abs(v64).sum()


def test_quantiser_chunk_partition_only_changes_rounding_order():
    """The per-chunk / across-chunk summation order is fixed; the result for a tensor split into
    chunks differs from numpy's pairwise fp64 sum by rounding only (codes identical here)."""
    rng = np.random.default_rng(11)
    v = rng.standard_normal(64 * 9).astype(np.float32)
    a = O.quantize_tensor(v, np.full(9, 64, np.int32))
    b = O.quantize_tensor(v, np.array([64 * 9], np.int32))
    assert np.array_equal(a[3], b[3])
    assert np.allclose(a[2], b[2], rtol=1e-6, atol=0)


def test_quantiser_shift_equivariance():
    rng = np.random.default_rng(12)
    v = (rng.integers(-50, 50, 256)).astype(np.float32)  # integers: shifts are exact
    cnt = np.array([64] * 4, np.int32)
    mu, sg, lut, code = O.quantize_tensor(v, cnt)
    mu2, sg2, lut2, code2 = O.quantize_tensor((v + np.float32(1024.0)).astype(np.float32), cnt)
    assert np.array_equal(code, code2) and sg == sg2
    used = np.unique(code)
    assert np.allclose(lut2[used], lut[used] + 1024.0, rtol=0, atol=1e-3)


# ----------------------------------------------------------------------------- packing

def test_pack_handworked_bytes():
    # two 12-bit indices 0x123, 0xABC little-endian bit order -> 23 C1 AB; codes 1,2 -> 0b1001 = 0x09
    rec = O.pack_record(np.array([0x123, 0xABC]), np.array([1, 2]), k=2)
    assert rec.size == 16 and O.record_stride(2) == 16
    assert list(rec[:3]) == [0x23, 0xC1, 0xAB]
    assert rec[3] == 0x09 and not rec[4:].any()
    # k = 4 -> 6 index bytes, code byte at 6: codes 1,2,3,0 -> 1 | 2<<2 | 3<<4 = 0x39
    rec = O.pack_record(np.array([1, 2, 3, 4095]), np.array([1, 2, 3, 0]), k=4)
    assert list(rec[:7]) == [0x01, 0x20, 0x00, 0x03, 0xF0, 0xFF, 0x39]
    # odd k: k = 3 -> ceil(36/8) = 5 index bytes, codes at byte 5; a short chunk (m = 2) leaves slot 2 zero
    rec = O.pack_record(np.array([7, 8]), np.array([3, 3]), k=3)
    assert list(rec[:6]) == [0x07, 0x80, 0x00, 0x00, 0x00, 0x0F]


@pytest.mark.parametrize("k", [1, 41, 64, 82, 123, 256, 257, 1000, 2048])
def test_pack_roundtrip_and_stride(k):
    rng = np.random.default_rng(k)
    idx = np.sort(rng.choice(4096, k, replace=False)).astype(np.int32)
    code = rng.integers(0, 4, k).astype(np.uint8)
    rec = O.pack_record(idx, code, k)
    want_stride = (math.ceil(12 * k / 8) + math.ceil(2 * k / 8) + 15) // 16 * 16
    assert rec.size == want_stride
    i2, c2 = O.unpack_record(rec, k, k)
    assert np.array_equal(i2, idx) and np.array_equal(c2, code)
    # bits beyond the two blocks are zero
    used = np.zeros(rec.size * 8, bool)
    used[:12 * k] = True
    cb = math.ceil(12 * k / 8) * 8
    used[cb:cb + 2 * k] = True
    bits = np.unpackbits(rec, bitorder="little").astype(bool)
    assert not (bits & ~used).any()


def test_strides_of_the_benchmark_ks():
    assert [O.record_stride(k) for k in (41, 64, 82, 123)] == [80, 112, 144, 224]


def test_payload_size_against_paper_accounting():
    g = read_kv(os.path.join(GOLD, "paper_printed_values.txt"))
    from paper_2508_15706_b200 import inputs as I
    # the tensor-list recipe reproduces the paper's parameter counts
    assert sum(t.numel for t in I.dense_transformer(1024, 9, 2688, 32000)) == g["params_178M"]
    m512 = I.dense_transformer(1536, 12, 5440, 32000)
    assert sum(t.numel for t in m512) == g["params_512M"]
    assert sum(t.numel for t in I.dense_transformer(2560, 24, 7680, 32000, kv_dim=640)) == g["params_2B"]
    N = g["params_512M"]

    def size_mb(density, idx_bits, val_bits):  # the paper's accounting: N * density * bits / 8
        return N * density * (idx_bits + val_bits) / 8 / 1e6

    # the accounting form reproduces Table 1 with the appendix's achieved index rates ...
    assert abs(size_mb(32 / 4096, g["achieved_bits_k32"], 2) - g["size_MB_sparseloco_density_0.78"]) < 0.006
    assert abs(size_mb(128 / 4096, g["achieved_bits_k128"], 2) - g["size_MB_sparseloco_density_3.12"]) < 0.006
    assert abs(size_mb(32 / 4096, g["naive_index_bits"], 8) - g["size_MB_demo_density_0.78"]) < 0.006
    assert abs(size_mb(128 / 4096, g["naive_index_bits"], 8) - g["size_MB_demo_density_3.12"]) < 0.006
    assert abs(N / 1e6 - g["size_MB_diloco_8bit"]) < 0.006
    # ... and the entropy bound the appendix quotes
    for k in (32, 128, 256):
        bound = math.log2(math.comb(4096, k)) / k
        assert abs(bound - g[f"bound_bits_k{k}"]) < 0.1
    # ... so with 12-bit indices and 2-bit codes the oracle's records must cost exactly
    # density * 14 / 8 bytes per parameter on the 2-D tensors (k = 64, 128: no padding)
    two_d = [t for t in m512 if t.rows > 1]
    for k in (64, 128, 256):
        cfg = O.Config(k=k)
        tab = O.Table([(t.rows, t.cols) for t in two_d])
        n2 = sum(t.numel for t in two_d)
        assert O.payload_bytes(cfg, tab) - 16 * len(two_d) == n2 * k * 14 // (4096 * 8)
    # whole model at k = 128: 28.02 MB + tables + the 25 short norm chunks
    cfg = O.Config(k=128)
    tab = O.Table([(t.rows, t.cols) for t in m512])
    assert abs(O.payload_bytes(cfg, tab) / 1e6 - size_mb(128 / 4096, 12, 2)) < 0.02


# ----------------------------------------------------------------------------- compression end to end

def small_problem(seed, shapes, R, scale=1e-3):
    rng = np.random.default_rng(seed)
    tab = O.Table(shapes)
    n = tab.numel
    theta = (rng.standard_normal(n) * 0.02).astype(np.float32)
    theta_r = [(theta - (rng.standard_t(3, n) * scale).astype(np.float32)).astype(np.float32) for _ in range(R)]
    e = [(rng.standard_normal(n) * scale).astype(np.float32) for _ in range(R)]
    return tab, theta, theta_r, e


def test_compress_error_feedback_invariant_and_density():
    shapes = [(128, 128), (1, 5000), (8, 1024), (1, 48)]
    tab, theta, theta_r, e = small_problem(3, shapes, 1)
    cfg = O.Config(k=64, beta=0.95)
    e_old = e[0].copy()
    u = O.ef_accumulate(theta, theta_r[0], e_old, 0.95)  # pinned above
    out = O.compress(cfg, tab, theta, theta_r[0], e[0])
    slots = O.total_slots(cfg, tab)
    assert slots == 64 * 4 + 64 * 2 + 64 * 2 + 48 == out.sel_idx.size
    # walk the slot lists, rebuild the dense decoded vector
    dense_hat = np.zeros_like(theta)
    selected = np.zeros(theta.size, bool)
    w = 0
    for j, (rows, cols, off) in enumerate(tab.shapes):
        for ch in range(O.num_chunks(cfg, tab, j)):
            L = O.chunk_len(cfg, tab, j, ch)
            m = min(64, L)
            pos = np.array([off + O.chunk_pos(cfg, tab, j, ch, int(p)) for p in out.sel_idx[w:w + m]])
            assert not selected[pos].any()
            selected[pos] = True
            dense_hat[pos] = out.sel_hat[w:w + m]
            assert np.array_equal(u[pos], out.sel_val[w:w + m])
            # the chunk's selection is the brute-force Top-k of u over that chunk
            allpos = np.array([off + O.chunk_pos(cfg, tab, j, ch, p) for p in range(L)])
            assert np.array_equal(brute_topk(u[allpos], 64), out.sel_idx[w:w + m])
            w += m
    assert w == slots
    # payload + new error = beta e_old + Delta:  exactly u where nothing was sent, u - hat (one fp32
    # rounding) where something was
    assert np.array_equal(e[0][~selected], u[~selected])
    assert np.array_equal(e[0][selected], (u[selected] - dense_hat[selected]).astype(np.float32))
    resid = e[0].astype(np.float64) + dense_hat.astype(np.float64) - u.astype(np.float64)
    assert np.all(np.abs(resid) <= np.spacing(np.abs(e[0])).astype(np.float64) * 0.5 + 1e-45)
    # decoded values come from the per-tensor table
    w = 0
    for j in range(tab.n):
        mj = sum(min(64, O.chunk_len(cfg, tab, j, ch)) for ch in range(O.num_chunks(cfg, tab, j)))
        assert set(np.unique(out.sel_hat[w:w + mj])) <= set(out.stats[j, 2:6])
        w += mj
    # payload decodes to the same sparse lists
    idx2, hat2 = O.decode_payload(cfg, tab, out.payload)
    assert np.array_equal(idx2, out.sel_idx) and np.array_equal(hat2, out.sel_hat)
    assert out.payload.size == 16 * 4 + 112 * (4 + 2 + 2 + 1)
    assert np.array_equal(out.payload[:16].view(np.float32), out.stats[0, 2:6])


def test_compress_freeze_and_zero_cases():
    shapes = [(64, 64), (1, 100)]
    tab, theta, theta_r, e = small_problem(4, shapes, 1)
    e_before = e[0].copy()
    out = O.compress(O.Config(k=8, ef_enabled=0), tab, theta, theta_r[0], e[0])
    assert np.array_equal(e[0], e_before)  # freeze: e untouched
    d = theta - theta_r[0]
    assert np.array_equal(out.sel_idx[:8], brute_topk(d[:4096], 8))
    # Delta = 0 and e = 0: everything stays zero, selection is the first k indices, all codes 3
    z = np.zeros_like(theta)
    ez = np.zeros_like(theta)
    out = O.compress(O.Config(k=8), tab, theta, theta.copy(), ez)
    assert not ez.any() and not out.sel_hat.any()
    assert list(out.sel_idx) == list(range(8)) * 2
    idx, code = O.unpack_record(out.payload[32:48].copy(), 8, 8)
    assert list(code) == [3] * 8
    # beta = 0: e_new = Delta - Delta_hat regardless of the old e
    e1 = e_before.copy()
    o1 = O.compress(O.Config(k=8, beta=0.0), tab, theta, theta_r[0], e1)
    e2 = np.zeros_like(e_before)
    o2 = O.compress(O.Config(k=8, beta=0.0), tab, theta, theta_r[0], e2)
    assert np.array_equal(e1, e2) and np.array_equal(o1.payload, o2.payload)


def test_error_shrinks_when_drift_stops():
    shapes = [(64, 128)]
    tab, theta, theta_r, e = small_problem(6, shapes, 1)
    cfg = O.Config(k=64, beta=0.9)
    O.compress(cfg, tab, theta, theta_r[0], e[0])
    prev = np.linalg.norm(e[0].astype(np.float64))
    for _ in range(3):
        O.compress(cfg, tab, theta, theta.copy(), e[0])  # Delta = 0
        cur = np.linalg.norm(e[0].astype(np.float64))
        assert cur <= 0.9 * prev * (1 + 1e-6)
        prev = cur


# ----------------------------------------------------------------------------- aggregate + outer update

def test_full_density_unquantised_is_parameter_averaging():
    """k = C, no quantiser, beta = 0, alpha = 1: theta_new = mean_r theta_r (the paper notes that
    100 % density is DiLoCo without outer momentum)."""
    shapes = [(64, 64), (1, 1000)]
    R = 4
    tab, theta, theta_r, e = small_problem(8, shapes, R)
    cfg = O.Config(k=4096, R=R, beta=0.0, outer_lr=1.0, quant_bits=32)
    outs = [O.compress(cfg, tab, theta, theta_r[r], e[r]) for r in range(R)]
    for r in range(R):
        assert not e[r].any()  # everything was sent
    th = theta.copy()
    O.aggregate_apply_sparse(cfg, tab, [o.sel_idx for o in outs], [o.sel_hat for o in outs], th)
    deltas = np.stack([(theta - t).astype(np.float32).astype(np.float64) for t in theta_r])
    want = theta.astype(np.float64) - deltas.mean(axis=0)
    assert np.max(np.abs(th.astype(np.float64) - want)) <= np.max(np.spacing(np.abs(th))) * 0.51
    avg = np.mean(np.stack(theta_r).astype(np.float64), axis=0)
    assert np.max(np.abs(th.astype(np.float64) - avg)) <= 4 * np.max(np.spacing(np.abs(theta)))
    # alpha = 0.5 moves half way
    cfg_h = O.Config(k=4096, R=R, beta=0.0, outer_lr=0.5, quant_bits=32)
    th2 = theta.copy()
    O.aggregate_apply_sparse(cfg_h, tab, [o.sel_idx for o in outs], [o.sel_hat for o in outs], th2)
    want2 = theta.astype(np.float64) - 0.5 * deltas.mean(axis=0)
    assert np.max(np.abs(th2.astype(np.float64) - want2)) <= np.max(np.spacing(np.abs(th2))) * 0.51


def test_aggregate_special_cases():
    shapes = [(128, 64), (1, 300)]
    R = 3
    tab, theta, theta_r, e = small_problem(9, shapes, R)
    cfg = O.Config(k=16, R=R)
    outs = [O.compress(cfg, tab, theta, theta_r[r], e[r]) for r in range(R)]
    payloads = [o.payload for o in outs]
    # alpha = 0: bit-unchanged
    th = theta.copy()
    O.aggregate_apply(O.Config(k=16, R=R, outer_lr=0.0), tab, payloads, th)
    assert np.array_equal(th, theta)
    # untouched positions bit-unchanged, touched ones follow the definition with divisor R
    th = theta.copy()
    O.aggregate_apply(cfg, tab, payloads, th)
    acc = np.zeros(theta.size, np.float64)
    hit = np.zeros(theta.size, bool)
    for o in outs:
        w = 0
        for j, (rows, cols, off) in enumerate(tab.shapes):
            for ch in range(O.num_chunks(cfg, tab, j)):
                m = min(16, O.chunk_len(cfg, tab, j, ch))
                for s in range(m):
                    pos = off + O.chunk_pos(cfg, tab, j, ch, int(o.sel_idx[w]))
                    acc[pos] += float(o.sel_hat[w])
                    hit[pos] = True
                    w += 1
    assert np.array_equal(th[~hit], theta[~hit])
    want = (theta.astype(np.float64) - acc / R).astype(np.float32)
    assert np.array_equal(th[hit], want[hit])
    # R identical workers: Delta equals one worker's decoded vector
    th = theta.copy()
    O.aggregate_apply(cfg, tab, [payloads[0]] * R, th)
    one = np.zeros(theta.size, np.float64)
    idx0, hat0 = O.decode_payload(cfg, tab, payloads[0])
    w = 0
    for j, (rows, cols, off) in enumerate(tab.shapes):
        for ch in range(O.num_chunks(cfg, tab, j)):
            m = min(16, O.chunk_len(cfg, tab, j, ch))
            for s in range(m):
                one[off + O.chunk_pos(cfg, tab, j, ch, int(idx0[w]))] = float(hat0[w])
                w += 1
    assert np.allclose(th.astype(np.float64), theta.astype(np.float64) - one, rtol=0, atol=1e-8)
    # absent worker: divisor stays R by default, becomes the present count on request
    th_r = theta.copy()
    O.aggregate_apply(cfg, tab, [payloads[0], None, payloads[2]], th_r)
    th_p = theta.copy()
    O.aggregate_apply(O.Config(k=16, R=R, divide_by_present=1), tab, [payloads[0], None, payloads[2]], th_p)
    moved = th_r != theta
    ratio = (th_p[moved].astype(np.float64) - theta[moved]) / (th_r[moved].astype(np.float64) - theta[moved])
    assert np.allclose(ratio, 1.5, rtol=1e-3)
    # no payload at all: nothing changes
    th = theta.copy()
    O.aggregate_apply(cfg, tab, [None] * R, th)
    assert np.array_equal(th, theta)


def test_outer_step_equals_compress_then_aggregate_and_resumes():
    shapes = [(64, 192), (1, 4100)]
    R = 2
    tab, theta, theta_r, e = small_problem(10, shapes, R)
    cfg = O.Config(k=32, R=R, outer_lr=0.7)
    th_a, e_a = theta.copy(), [x.copy() for x in e]
    pa = O.outer_step(cfg, tab, th_a, theta_r, e_a)
    th_b, e_b = theta.copy(), [x.copy() for x in e]
    pb = [O.compress(cfg, tab, th_b, theta_r[r], e_b[r]).payload for r in range(R)]
    O.aggregate_apply(cfg, tab, pb, th_b)
    assert np.array_equal(th_a, th_b)
    for r in range(R):
        assert np.array_equal(e_a[r], e_b[r]) and np.array_equal(pa[r], pb[r])
    # state is (theta, e): continuing from copies gives the same second step
    rng = np.random.default_rng(0)
    theta_r2 = [(th_a - (rng.standard_normal(th_a.size) * 1e-3).astype(np.float32)).astype(np.float32) for _ in range(R)]
    th_c, e_c = th_a.copy(), [x.copy() for x in e_a]
    p1 = O.outer_step(cfg, tab, th_a, theta_r2, e_a)
    p2 = O.outer_step(cfg, tab, th_c, theta_r2, e_c)
    assert np.array_equal(th_a, th_c) and all(np.array_equal(a, b) for a, b in zip(p1, p2))


def test_threads_do_not_change_results():
    shapes = [(128, 128), (1, 9000)]
    tab, theta, theta_r, e = small_problem(13, shapes, 1)
    cfg = O.Config(k=64)
    e1, e2 = e[0].copy(), e[0].copy()
    O.set_threads(1)
    a = O.compress(cfg, tab, theta, theta_r[0], e1)
    O.set_threads(4)
    b = O.compress(cfg, tab, theta, theta_r[0], e2)
    O.set_threads(1)
    assert np.array_equal(a.payload, b.payload) and np.array_equal(e1, e2)
