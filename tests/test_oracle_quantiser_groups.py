"""Pins for the oracle's quantiser beyond one 64-chunk summation group.

Sec. 4 fixes the statistics (mean, sigma, centroid table) but not the order of the sums; the
reading taken is fp64 in three levels, each left to right: slots of a chunk, chunks of a group of
64 consecutive chunks, groups.  Two independent checks, on tensors of 65 to 16,000 chunks with
uneven per-chunk counts and a short last group:

(a) an independent restatement of that order as plain Python loops over lists (Python floats are
    IEEE doubles), compared bit for bit on inputs whose sums depend strongly on the order (huge
    dynamic range, mixed signs).  The same restatement with another group size, or with one flat
    chain, must DIFFER on those inputs, which shows that the comparison sees the grouping.
(b) exact arithmetic on benign inputs: every fp32 output equals the correctly rounded exact value
    (mean, population sigma of the fp32-centred values, per-bin means), or is one ulp from it in a
    small number of cases.  This is what the method defines whatever the order.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle as O

GROUP = 64
CHUNKS = (65, 130, 2049, 16000)


def f32(x: float) -> float:
    """Round a Python float to fp32 (nearest even), returned as a Python float."""
    return float(np.float32(x))


def restated(v, cnt, group):
    """mu, sigma, table, codes by the three-level order written out with lists and loops."""
    v = [float(x) for x in v]
    cnt = [int(c) for c in cnt]
    n = sum(cnt)
    starts, pos = [], 0
    for c in cnt:
        starts.append(pos)
        pos += c

    def three_level(term, lanes=1, which=None):
        total = [0.0] * lanes
        for g0 in range(0, len(cnt), group):
            gsum = [0.0] * lanes
            for c in range(g0, min(g0 + group, len(cnt))):
                csum = [0.0] * lanes
                for s in range(cnt[c]):
                    i = starts[c] + s
                    lane = 0 if which is None else which[i]
                    csum[lane] = csum[lane] + term(i)
                for b in range(lanes):
                    gsum[b] = gsum[b] + csum[b]
            for b in range(lanes):
                total[b] = total[b] + gsum[b]
        return total

    with np.errstate(all="ignore"):
        mu = f32(three_level(lambda i: v[i])[0] / n)
        cen = [f32(x - mu) for x in v]
        sigma = f32(math.sqrt(three_level(lambda i: cen[i] * cen[i])[0] / n))
        t = f32(3.0 * sigma)
        code = [int(c >= -t) + int(c >= 0.0) + int(c >= t) for c in cen]
        sums = three_level(lambda i: v[i], lanes=4, which=code)
    cnts = [code.count(b) for b in range(4)]
    lut = [f32(sums[b] / cnts[b]) if cnts[b] else 0.0 for b in range(4)]
    return mu, sigma, lut, code


def bits(x) -> int:
    return int(np.array([x], np.float32).view(np.uint32)[0])


def order_sensitive_values(rng, n):
    """fp32 values over ~100 binades, every one accompanied somewhere by its exact negation: the
    exact sum is 0 and what an fp64 chain returns is made of the small terms that survive between a
    large term and its opposite, i.e. it depends on the order far above fp32 resolution."""
    h = n // 2
    e = rng.integers(-10, 90, h)
    m = 1.0 + rng.integers(0, 1 << 10, h) / float(1 << 10)
    s = rng.choice([-1.0, 1.0], h)
    half = (s * m * np.exp2(e.astype(np.float64))).astype(np.float32)
    v = np.concatenate([half, -half, np.ones(n - 2 * h, np.float32)])
    return v[rng.permutation(n)]


@pytest.mark.parametrize("n_chunks", CHUNKS)
def test_three_level_order_bit_for_bit(n_chunks):
    rng = np.random.default_rng(1000 + n_chunks)
    kmax = 64 if n_chunks <= 2049 else 16
    cnt = rng.integers(1, kmax + 1, n_chunks).astype(np.int32)
    v = order_sensitive_values(rng, int(cnt.sum()))
    mu, sigma, lut, code = O.quantize_tensor(v, cnt)
    r_mu, r_sigma, r_lut, r_code = restated(v, cnt, GROUP)
    assert bits(mu) == bits(r_mu)
    assert bits(sigma) == bits(r_sigma)
    assert [bits(x) for x in lut] == [bits(x) for x in r_lut]
    assert list(code) == r_code


@pytest.mark.parametrize("n_chunks,others", ((65, (32,)), (130, (32, 128, 1 << 30)), (2049, (32, 128, 1 << 30))))
def test_the_comparison_sees_the_grouping(n_chunks, others):
    """With groups of 32, groups of 128 or one flat chain the restatement no longer matches the
    oracle on these inputs: a change of the group size (or a lost carry between groups) is visible.
    (65 chunks = one full group and a group of one chunk, which a flat chain over the chunks adds in
    the same order: only the smaller group size differs there.)"""
    rng = np.random.default_rng(1000 + n_chunks)
    cnt = rng.integers(1, 65, n_chunks).astype(np.int32)
    v = order_sensitive_values(rng, int(cnt.sum()))
    mu, sigma, lut, code = O.quantize_tensor(v, cnt)
    got = (bits(mu), bits(sigma), tuple(bits(x) for x in lut))
    for other in others:
        o_mu, o_sigma, o_lut, _ = restated(v, cnt, other)
        assert (bits(o_mu), bits(o_sigma), tuple(bits(x) for x in o_lut)) != got, other


def nearest_f32(x: Fraction) -> np.float32:
    g = np.float32(float(x))
    best, best_d = g, abs(Fraction(float(g)) - x)
    for c in (np.nextafter(g, np.float32(np.inf)), np.nextafter(g, np.float32(-np.inf))):
        d = abs(Fraction(float(c)) - x)
        if d < best_d:
            best, best_d = c, d
    return best


def ulps_apart(a, b) -> int:
    return abs(int(np.array([a], np.float32).view(np.int32)[0]) - int(np.array([b], np.float32).view(np.int32)[0]))


@pytest.mark.parametrize("n_chunks", CHUNKS)
def test_outputs_are_the_correctly_rounded_exact_statistics(n_chunks):
    rng = np.random.default_rng(2000 + n_chunks)
    kmax = 64 if n_chunks <= 2049 else 8
    cnt = rng.integers(1, kmax + 1, n_chunks).astype(np.int32)
    n = int(cnt.sum())
    v = (rng.standard_t(4, n) * 3e-3 + 1e-3).astype(np.float32)
    mu, sigma, lut, code = O.quantize_tensor(v, cnt)

    exact = [Fraction(float(x)) for x in v]
    mu_exact = sum(exact, Fraction(0)) / n
    one_ulp = 0
    d = ulps_apart(mu, nearest_f32(mu_exact))
    assert d <= 1
    one_ulp += d
    # sigma and the codes are defined on the values centred by the fp32 mean that was actually taken
    cen = (v - mu).astype(np.float32)
    var_exact = sum((Fraction(float(c)) ** 2 for c in cen), Fraction(0)) / n
    # sqrt of a rational: bracket the fp32 candidate by exact squares
    s_guess = np.float32(math.sqrt(float(var_exact)))
    lo, hi = np.nextafter(s_guess, np.float32(0)), np.nextafter(s_guess, np.float32(np.inf))
    cands = sorted({float(lo), float(s_guess), float(hi)})
    best = min(cands, key=lambda c: abs(Fraction(c) ** 2 - var_exact) / (Fraction(c) + Fraction(float(s_guess))))
    d = ulps_apart(sigma, np.float32(best))
    assert d <= 1
    one_ulp += d
    t = np.float32(3.0) * sigma
    want_code = (cen >= -t).astype(int) + (cen >= 0).astype(int) + (cen >= t).astype(int)
    assert np.array_equal(code, want_code)
    for b in range(4):
        m = code == b
        if not m.any():
            assert bits(lut[b]) == 0
            continue
        cb = sum((exact[i] for i in np.nonzero(m)[0]), Fraction(0)) / int(m.sum())
        d = ulps_apart(lut[b], nearest_f32(cb))
        assert d <= 1
        one_ulp += d
    assert one_ulp <= 1, one_ulp
