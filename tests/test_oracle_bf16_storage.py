"""Pins for the oracle's bfloat16-storage mode (the paper is silent on storage types; the reading: all
arithmetic as in the fp32 mode on the widened values, every store rounded once to the nearest bfloat16,
ties to even).  The rounding routine is pinned against hand-worked cases, torch's fp32 -> bf16 cast and
an exact-rational nearest search; the mode itself against the fp32 mode followed by torch's cast (for
e, whose stored value is a single fp32 result) and against the exact-rational search (for theta, whose
stored value rounds an fp64 expression)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle as O


def _torch_bf16(a: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def _is_bf16(a: np.ndarray) -> bool:
    return not np.any(np.ascontiguousarray(a, np.float32).view(np.uint32) & np.uint32(0xFFFF))


def _nearest_bf16_exact(x: float) -> float:
    """Nearest bfloat16 to the real number x by exact rational arithmetic: the two neighbours on the
    bfloat16 grid around x are found from the fp32 truncation, the closer wins, the even one on a tie."""
    if x == 0.0:
        return x
    s = -1.0 if x < 0 else 1.0
    fx = Fraction(abs(x))
    lo_bits = np.array([abs(x)], np.float64).astype(np.float32)
    # truncate towards zero on the bf16 grid, then correct if fp32 rounding went above |x|
    b = int(lo_bits.view(np.uint32)[0]) & 0xFFFF0000
    lo = np.array([b], np.uint32).view(np.float32)[0]
    if Fraction(float(lo)) > fx:
        b -= 0x10000
        lo = np.array([b], np.uint32).view(np.float32)[0]
    hi = np.array([b + 0x10000], np.uint32).view(np.float32)[0]
    dl, dh = fx - Fraction(float(lo)), Fraction(float(hi)) - fx
    if dl < dh:
        r = lo
    elif dh < dl:
        r = hi
    else:
        r = lo if ((b >> 16) & 1) == 0 else hi
    return s * float(r)


def test_bf16_round_handworked():
    # spacing of bfloat16 in [1, 2) is 2^-7
    assert O.bf16_round(1.0 + 2.0 ** -8) == 1.0                       # tie -> even (1.0)
    assert O.bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6       # tie -> even (1 + 2/128)
    assert O.bf16_round(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert O.bf16_round(-(1.0 + 2.0 ** -8 + 2.0 ** -20)) == -(1.0 + 2.0 ** -7)
    assert O.bf16_round(3.140625) == 3.140625                          # 11.001001b: 8 significant bits
    assert O.bf16_round(0.1) == 0.10009765625                          # 0x3DCD -> 0x3DCD0000
    # subnormals: spacing 2^-133
    assert O.bf16_round(0.5 * 2.0 ** -133) == 0.0                      # tie -> even (0)
    assert O.bf16_round(1.5 * 2.0 ** -133) == 2.0 ** -132              # tie -> even (2 steps)
    assert O.bf16_round(0.75 * 2.0 ** -133) == 2.0 ** -133
    assert np.signbit(O.bf16_round(-0.0)) and O.bf16_round(-0.0) == 0.0
    # one rounding from a double, not two: the fp32 detour would land on the tie and fall to 1.0
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert float(np.float32(x)) == 1.0 + 2.0 ** -8
    assert O.bf16_round_d(x) == 1.0 + 2.0 ** -7


def test_bf16_round_against_torch_cast_and_exact_search():
    rng = np.random.default_rng(5)
    a = np.concatenate([
        rng.standard_normal(4000).astype(np.float32),
        (rng.standard_normal(500) * 1e-39).astype(np.float32),                 # denormals
        (rng.standard_normal(500) * 1e30).astype(np.float32),
        (rng.integers(0, 1 << 16, 2000).astype(np.uint32) << 16 | 0x8000).view(np.float32),  # exact ties
        (rng.integers(0, 1 << 16, 2000).astype(np.uint32) << 16 | 0x7FFF).view(np.float32),
        (rng.integers(0, 1 << 16, 2000).astype(np.uint32) << 16 | 0x8001).view(np.float32),
    ])
    a = a[np.isfinite(a) & (np.abs(a) < 3e38)]
    got = np.array([O.bf16_round(float(x)) for x in a], np.float32)
    assert np.array_equal(got.view(np.uint32), _torch_bf16(a).view(np.uint32))
    assert _is_bf16(got)
    d = rng.standard_normal(400) * np.exp(rng.uniform(-60, 60, 400))
    for x in d:
        assert O.bf16_round_d(float(x)) == _nearest_bf16_exact(float(x)), x


SHAPES = [(128, 128), (1, 5000), (64, 192), (1, 40)]


def _inputs(seed, R):
    rng = np.random.default_rng(seed)
    tab = O.Table(SHAPES)
    n = tab.numel
    theta = _torch_bf16(rng.standard_normal(n).astype(np.float32) * 0.05)
    local = [_torch_bf16(theta + rng.standard_t(4, n).astype(np.float32) * 1e-3) for _ in range(R)]
    e = [_torch_bf16(rng.standard_t(4, n).astype(np.float32) * 5e-4) for _ in range(R)]
    return tab, theta, local, e


@pytest.mark.parametrize("bits,k", [(2, 64), (2, 7), (4, 33)])
def test_compress_rounds_only_the_store(bits, k):
    """Selection, quantiser and payload see the unrounded u: the payload equals the fp32 mode's, and the
    stored e is the fp32 mode's e pushed through torch's bf16 cast."""
    tab, theta, local, e = _inputs(10 + k, 2)
    for r in range(2):
        e32, e16 = e[r].copy(), e[r].copy()
        a = O.compress(O.Config(k=k, R=2, beta=0.9, quant_bits=bits), tab, theta, local[r], e32)
        b = O.compress(O.Config(k=k, R=2, beta=0.9, quant_bits=bits, storage_bf16=1), tab, theta, local[r], e16)
        assert np.array_equal(a.payload, b.payload)
        assert np.array_equal(a.sel_val.view(np.uint32), b.sel_val.view(np.uint32))
        assert _is_bf16(e16) and not _is_bf16(e32)
        assert np.array_equal(e16.view(np.uint32), _torch_bf16(e32).view(np.uint32))
    # the freeze leaves e alone in this mode too
    e16 = e[0].copy()
    O.compress(O.Config(k=k, R=2, beta=0.9, quant_bits=bits, storage_bf16=1, ef_enabled=0), tab, theta, local[0], e16)
    assert np.array_equal(e16, e[0])


def test_update_is_the_nearest_bf16_of_the_fp64_expression():
    R, k = 3, 16
    tab, theta, local, e = _inputs(77, R)
    cfg = O.Config(k=k, R=R, beta=0.9, outer_lr=0.7, storage_bf16=1)
    pays, lists = [], []
    for r in range(R):
        out = O.compress(cfg, tab, theta, local[r], e[r])
        pays.append(out.payload)
        lists.append((out.sel_idx, out.sel_hat))
    th = theta.copy()
    O.aggregate_apply(cfg, tab, pays, th)
    assert _is_bf16(th)
    # the fp64 expression, element by element, from the decoded lists (positions through the oracle's geometry)
    acc = np.zeros(tab.numel, np.float64)
    hit = np.zeros(tab.numel, bool)
    for r in range(R):
        idx, hat = lists[r]
        w = 0
        for j in range(tab.n):
            for ch in range(O.num_chunks(cfg, tab, j)):
                m = min(k, O.chunk_len(cfg, tab, j, ch))
                for s in range(m):
                    pos = tab.shapes[j][2] + O.chunk_pos(cfg, tab, j, ch, int(idx[w]))
                    acc[pos] += float(hat[w])
                    hit[pos] = True
                    w += 1
    assert np.array_equal(th[~hit], theta[~hit])          # untouched elements keep their bits
    x = theta.astype(np.float64) - 0.7 * acc / R
    pick = np.nonzero(hit)[0]
    for i in pick[:: max(1, pick.size // 600)]:
        assert float(th[i]) == _nearest_bf16_exact(float(x[i])), i
    assert np.count_nonzero(th[hit] != theta[hit]) > 0.2 * pick.size   # the step does move parameters


def test_fp32_mode_is_untouched_by_the_new_field():
    tab, theta, local, e = _inputs(3, 1)
    e0 = e[0].copy()
    a = O.compress(O.Config(k=9, R=1, beta=0.5), tab, theta, local[0], e0)
    assert not _is_bf16(e0) and a.payload.size == O.payload_bytes(O.Config(k=9), tab)
