"""Pins for the oracle's entropy-coded index format (App. "Compression of indices"): a hand-worked
stream, an independent bit-by-bit Python implementation of the definition, the closed-form worst
case, and the rate on uniformly drawn index sets between the information-theoretic bound and the
rates the paper reports (8.9 / 6.6 / 5.6 bits per value at k = 32 / 128 / 256, C = 4096)."""
import math
import os

import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "index_codec_handworked.txt")


# ---- the definition, written independently of the C code (lists of bits, no packing tricks)

def divisor(L, m):
    return max(1, (693 * (L - m) + 500 * (m + 1)) // (1000 * (m + 1)))


def py_encode(idx, L):
    m = len(idx)
    M = divisor(L, m)
    b = max(0, math.ceil(math.log2(M))) if M > 1 else 0
    cut = (1 << b) - M
    bits, prev = [], -1
    for p in idx:
        g = p - prev - 1
        prev = p
        q, r = divmod(g, M)
        bits += [1] * q + [0]
        if M > 1:
            if r < cut:
                bits += [int(c) for c in format(r, "b").zfill(b - 1)] if b > 1 else []
            else:
                bits += [int(c) for c in format(r + cut, "b").zfill(b)]
    return bits


def py_decode(bits, m, L):
    M = divisor(L, m)
    b = max(0, math.ceil(math.log2(M))) if M > 1 else 0
    cut = (1 << b) - M
    out, prev, i = [], -1, 0
    for _ in range(m):
        q = 0
        while bits[i]:
            q += 1
            i += 1
        i += 1
        r = 0
        if M > 1:
            for _ in range(b - 1):
                r = 2 * r + bits[i]
                i += 1
            if r >= cut:
                r = 2 * r + bits[i] - cut
                i += 1
        prev = prev + 1 + q * M + r
        out.append(prev)
    return out, i


def unpack_bits(stream, n):
    return [(int(stream[i >> 3]) >> (i & 7)) & 1 for i in range(n)]


def test_handworked_streams():
    txt = open(GOLD).read()
    stream, n = O.ixc_encode_chunk(np.array([1, 5, 6], np.int32), 16)
    assert n == 7 and stream[0] == 22
    assert "nbits = 7" in txt and "byte0 = 22" in txt
    stream, n = O.ixc_encode_chunk(np.array([100, 4095], np.int32), 4096)
    want = [int(c) for c in "0" + "0010110010" + "11110" + "0100100000"]
    assert n == 26 and unpack_bits(stream, n) == want
    assert "bits2 = 0 0010110010 11110 0100100000" in txt


@pytest.mark.parametrize("L,k", [(16, 1), (16, 3), (16, 16), (64, 5), (700, 41), (4096, 1), (4096, 32), (4096, 64),
                                 (4096, 123), (4096, 256), (2048, 64), (40, 64)])
def test_oracle_matches_independent_definition_and_round_trips(L, k):
    rng = np.random.default_rng(1000 * L + k)
    m = min(k, L)
    for trial in range(30):
        if trial == 0:
            idx = np.arange(m)                      # all at the start: every gap 0
        elif trial == 1:
            idx = np.arange(L - m, L)               # all at the end: one huge gap
        else:
            idx = np.sort(rng.choice(L, m, replace=False))
        idx = idx.astype(np.int32)
        stream, n = O.ixc_encode_chunk(idx, L)
        bits = py_encode(list(map(int, idx)), L)
        assert n == len(bits) and unpack_bits(stream, n) == bits
        back, used = O.ixc_decode_chunk(stream, m, L)
        assert used == n and np.array_equal(back, idx)
        assert py_decode(bits, m, L) == (list(map(int, idx)), n)
        # closed-form worst case: one zero-bit and at most b remainder bits per value, and the
        # quotients together cannot exceed (L - m) / M
        M = divisor(L, m)
        b = math.ceil(math.log2(M)) if M > 1 else 0
        assert n <= m * (b + 1) + (L - m) // M


@pytest.mark.parametrize("k,paper,bound", [(32, 8.9, 8.318), (128, 6.6, 6.382), (256, 5.6, 5.376)])
def test_rate_between_bound_and_the_papers_rates(k, paper, bound):
    """Uniform index sets (the case the bound log2 C(4096, k) / k is about)."""
    assert abs(math.log2(math.comb(4096, k)) / k - bound) < 2e-3
    rng = np.random.default_rng(k)
    tot = 0
    n_chunks = 400
    for _ in range(n_chunks):
        idx = np.sort(rng.choice(4096, k, replace=False)).astype(np.int32)
        tot += O.ixc_encode_chunk(idx, 4096)[1]
    rate = tot / (n_chunks * k)
    assert bound <= rate <= paper, rate


def test_payload_round_trip_and_size():
    rng = np.random.default_rng(5)
    shapes = [(128, 192), (1, 5000), (1, 40), (64, 64), (1, 4096 * 20 + 7)]
    tab = O.Table(shapes)
    for k in (8, 41, 64):
        cfg = O.Config(k=k)
        n = tab.numel
        theta = rng.standard_normal(n).astype(np.float32)
        local = (theta - 1e-3 * rng.standard_normal(n)).astype(np.float32)
        e = np.zeros(n, np.float32)
        pay = O.compress(cfg, tab, theta, local, e).payload
        coded = O.ixc_encode_payload(cfg, tab, pay)
        assert coded.size % 16 == 0 and coded.size < pay.size
        assert np.array_equal(O.ixc_decode_payload(cfg, tab, coded), pay)
        # tables and code blocks are copied verbatim
        T, G = len(shapes), O.total_chunks(cfg, tab)
        assert np.array_equal(coded[:16 * T], pay[:16 * T])
        cb, ib, stride = (2 * k + 7) // 8, (12 * k + 7) // 8, O.record_stride(k)
        for g in (0, 1, G - 1):
            rec = pay[16 * T + g * stride:16 * T + (g + 1) * stride]
            assert np.array_equal(coded[16 * T + g * cb:16 * T + (g + 1) * cb], rec[ib:ib + cb])
        # directory: first entry 0, entries ascending
        doff = (16 * T + cb * G + 3) // 4 * 4
        d = coded[doff:doff + 4 * ((G + 15) // 16)].view(np.uint32)
        assert d[0] == 0 and np.all(np.diff(d.astype(np.int64)) > 0)
