"""ctypes access to the CPU oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.  The C source is
compiled with gcc on first use (or by `build()`), without fast-math and with
floating-point contraction off, so that every fp32 operation rounds once.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparseloco_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_sparseloco.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Tensor(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("offset", C.c_int64)]


class _Config(C.Structure):
    _fields_ = [("chunk_elems", C.c_int32), ("tile_dim", C.c_int32), ("k", C.c_int32),
                ("R", C.c_int32), ("H", C.c_int32), ("beta", C.c_float), ("outer_lr", C.c_float),
                ("quant_bits", C.c_int32), ("ef_enabled", C.c_int32),
                ("divide_by_present", C.c_int32), ("storage_bf16", C.c_int32)]


@dataclass
class Config:
    k: int
    R: int = 1
    H: int = 1
    beta: float = 0.95
    outer_lr: float = 1.0
    chunk_elems: int = 4096
    tile_dim: int = 64
    quant_bits: int = 2
    ef_enabled: int = 1
    divide_by_present: int = 0
    storage_bf16: int = 0   # 1: theta, theta_r, e hold bfloat16 values (as fp32 arrays); stores are rounded

    def c(self) -> _Config:
        return _Config(self.chunk_elems, self.tile_dim, self.k, self.R, self.H, self.beta,
                       self.outer_lr, self.quant_bits, self.ef_enabled, self.divide_by_present,
                       self.storage_bf16)


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        P = C.c_void_p
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_get_threads.restype = C.c_int
        for nm in ("orc_num_chunks",):
            getattr(L, nm).restype = C.c_int64
            getattr(L, nm).argtypes = [P, P]
        L.orc_chunk_len.restype = C.c_int64
        L.orc_chunk_len.argtypes = [P, P, C.c_int64]
        L.orc_chunk_pos.restype = C.c_int64
        L.orc_chunk_pos.argtypes = [P, P, C.c_int64, C.c_int64]
        for nm in ("orc_total_chunks", "orc_total_slots", "orc_payload_bytes"):
            getattr(L, nm).restype = C.c_int64
            getattr(L, nm).argtypes = [P, P, C.c_int32]
        L.orc_record_stride.restype = C.c_int64
        L.orc_record_stride.argtypes = [C.c_int32]
        L.orc_bf16_round.restype = C.c_float
        L.orc_bf16_round.argtypes = [C.c_float]
        L.orc_bf16_round_d.restype = C.c_float
        L.orc_bf16_round_d.argtypes = [C.c_double]
        L.orc_ef_accumulate.argtypes = [P, P, P, C.c_int64, C.c_float, C.c_int, P]
        L.orc_topk_chunk.restype = C.c_int32
        L.orc_topk_chunk.argtypes = [P, C.c_int32, C.c_int32, P]
        L.orc_quantize_tensor.argtypes = [P, P, C.c_int64, P, P, P, P]
        L.orc_quantize_tensor_q.argtypes = [P, P, C.c_int64, C.c_int32, P, P, P, P]
        L.orc_record_stride_q.restype = C.c_int64
        L.orc_record_stride_q.argtypes = [C.c_int32, C.c_int32]
        L.orc_header_bytes.restype = C.c_int64
        L.orc_header_bytes.argtypes = [C.c_int32]
        L.orc_pack_record_q.argtypes = [P, P, C.c_int32, C.c_int32, C.c_int32, P]
        L.orc_unpack_record_q.argtypes = [P, C.c_int32, C.c_int32, C.c_int32, P, P]
        L.orc_pack_record.argtypes = [P, P, C.c_int32, C.c_int32, P]
        L.orc_unpack_record.argtypes = [P, C.c_int32, C.c_int32, P, P]
        L.orc_compress.argtypes = [P, P, C.c_int32, P, P, P, P, P, P, P, P]
        L.orc_aggregate_apply_sparse.argtypes = [P, P, C.c_int32, P, P, P]
        L.orc_decode_payload.argtypes = [P, P, C.c_int32, P, P, P]
        L.orc_aggregate_apply.argtypes = [P, P, C.c_int32, P, P]
        L.orc_outer_step.argtypes = [P, P, C.c_int32, P, P, P, P]
        L.orc_diloco_step.argtypes = [P, C.c_int32, C.c_int32, C.c_float, C.c_float, P, P, P]
        L.orc_diloco_lom_step.argtypes = [P, C.c_int32, C.c_int32, C.c_float, C.c_float, P, P, P]
        L.orc_lom_step.argtypes = [P, P, C.c_int32, C.c_float, C.c_int32, P, P, P]
        L.orc_diloco_topk_step.argtypes = [P, P, C.c_int32, C.c_float, P, P, P, P]
        L.orc_lom_topk_step.argtypes = [P, P, C.c_int32, C.c_float, P, P, P, P]
        L.orc_ixc_encode_chunk.argtypes = [P, C.c_int32, C.c_int32, P, P]
        L.orc_ixc_decode_chunk.argtypes = [P, P, C.c_int32, C.c_int32, P]
        L.orc_ixc_encode_payload.argtypes = [P, P, C.c_int32, P, P]
        L.orc_ixc_encode_payload.restype = C.c_int64
        L.orc_ixc_decode_payload.argtypes = [P, P, C.c_int32, P, P]
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().orc_set_threads(int(n))


def get_threads() -> int:
    return lib().orc_get_threads()


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a: np.ndarray, dt) -> np.ndarray:
    assert a.dtype == dt and a.flags["C_CONTIGUOUS"], (a.dtype, dt)
    return a


class Table:
    """Tensor table (rows, cols, element offset) as the oracle sees it."""

    def __init__(self, shapes: Sequence[Sequence[int]], offsets: Optional[Sequence[int]] = None):
        n = len(shapes)
        self.n = n
        self.arr = (_Tensor * n)()
        pos = 0
        self.shapes = []
        for j, sh in enumerate(shapes):
            rows, cols = (1, sh[0]) if len(sh) == 1 else (sh[0], sh[1])
            off = offsets[j] if offsets is not None else pos
            self.arr[j] = _Tensor(rows, cols, off)
            self.shapes.append((rows, cols, off))
            pos = off + rows * cols
        self.numel = max((o + r * c for r, c, o in self.shapes), default=0)

    def ref(self):
        return C.cast(self.arr, C.c_void_p)

    def one(self, j: int):
        return C.cast(C.byref(self.arr[j]), C.c_void_p)


def num_chunks(cfg: Config, tab: Table, j: int) -> int:
    c = cfg.c()
    return lib().orc_num_chunks(C.byref(c), tab.one(j))


def chunk_len(cfg: Config, tab: Table, j: int, ch: int) -> int:
    c = cfg.c()
    return lib().orc_chunk_len(C.byref(c), tab.one(j), ch)


def chunk_pos(cfg: Config, tab: Table, j: int, ch: int, p: int) -> int:
    c = cfg.c()
    return lib().orc_chunk_pos(C.byref(c), tab.one(j), ch, p)


def total_chunks(cfg: Config, tab: Table) -> int:
    c = cfg.c()
    return lib().orc_total_chunks(C.byref(c), tab.ref(), tab.n)


def total_slots(cfg: Config, tab: Table) -> int:
    c = cfg.c()
    return lib().orc_total_slots(C.byref(c), tab.ref(), tab.n)


def payload_bytes(cfg: Config, tab: Table) -> int:
    c = cfg.c()
    return lib().orc_payload_bytes(C.byref(c), tab.ref(), tab.n)


def record_stride(k: int) -> int:
    return lib().orc_record_stride(k)


def ef_accumulate(theta, theta_r, e, beta: float, ef_enabled: int = 1) -> np.ndarray:
    u = np.empty_like(theta)
    lib().orc_ef_accumulate(_ptr(_chk(theta, np.float32)), _ptr(_chk(theta_r, np.float32)),
                            _ptr(_chk(e, np.float32)), theta.size, beta, ef_enabled, _ptr(u))
    return u


def topk_chunk(u: np.ndarray, k: int) -> np.ndarray:
    _chk(u, np.float32)
    out = np.empty(max(min(k, u.size), 1), dtype=np.int32)
    m = lib().orc_topk_chunk(_ptr(u), u.size, k, _ptr(out))
    return out[:m]


def quantize_tensor(v: np.ndarray, cnt: np.ndarray):
    """Returns (mu, sigma, lut[4], codes) for one tensor's selected values."""
    _chk(v, np.float32)
    cnt = np.ascontiguousarray(cnt, dtype=np.int32)
    mu = np.zeros(1, np.float32)
    sg = np.zeros(1, np.float32)
    lut = np.zeros(4, np.float32)
    code = np.zeros(max(v.size, 1), np.uint8)
    lib().orc_quantize_tensor(_ptr(v), _ptr(cnt), cnt.size, _ptr(mu), _ptr(sg), _ptr(lut), _ptr(code))
    return mu[0], sg[0], lut, code[:v.size]


def quantize_tensor_q(v: np.ndarray, cnt: np.ndarray, bits: int):
    """(mu, sigma, table[2^bits], codes) of the quantiser at `bits` bits per value."""
    _chk(v, np.float32)
    cnt = np.ascontiguousarray(cnt, dtype=np.int32)
    mu = np.zeros(1, np.float32)
    sg = np.zeros(1, np.float32)
    lut = np.zeros(16, np.float32)
    code = np.zeros(max(v.size, 1), np.uint8)
    lib().orc_quantize_tensor_q(_ptr(v), _ptr(cnt), cnt.size, bits, _ptr(mu), _ptr(sg), _ptr(lut), _ptr(code))
    return mu[0], sg[0], lut[:1 << bits], code[:v.size]


def record_stride_q(k: int, bits: int) -> int:
    return lib().orc_record_stride_q(k, bits)


def header_bytes(bits: int) -> int:
    return lib().orc_header_bytes(bits)


def pack_record_q(idx: np.ndarray, code: np.ndarray, k: int, bits: int) -> np.ndarray:
    idx = np.ascontiguousarray(idx, np.int32)
    code = np.ascontiguousarray(code, np.uint8)
    rec = np.zeros(record_stride_q(k, bits), np.uint8)
    lib().orc_pack_record_q(_ptr(idx), _ptr(code), idx.size, k, bits, _ptr(rec))
    return rec


def unpack_record_q(rec: np.ndarray, m: int, k: int, bits: int):
    idx = np.zeros(max(m, 1), np.int32)
    code = np.zeros(max(m, 1), np.uint8)
    lib().orc_unpack_record_q(_ptr(_chk(rec, np.uint8)), m, k, bits, _ptr(idx), _ptr(code))
    return idx[:m], code[:m]


def pack_record(idx: np.ndarray, code: np.ndarray, k: int) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    code = np.ascontiguousarray(code, dtype=np.uint8)
    rec = np.empty(record_stride(k), np.uint8)
    lib().orc_pack_record(_ptr(idx), _ptr(code), idx.size, k, _ptr(rec))
    return rec


def unpack_record(rec: np.ndarray, m: int, k: int):
    _chk(rec, np.uint8)
    idx = np.empty(max(m, 1), np.int32)
    code = np.empty(max(m, 1), np.uint8)
    lib().orc_unpack_record(_ptr(rec), m, k, _ptr(idx), _ptr(code))
    return idx[:m], code[:m]


@dataclass
class Compressed:
    payload: Optional[np.ndarray]
    sel_idx: np.ndarray
    sel_val: np.ndarray
    sel_hat: np.ndarray
    stats: np.ndarray  # per tensor: mu, sigma, the table (2^bits entries, then zeros up to 16)


def compress(cfg: Config, tab: Table, theta: np.ndarray, theta_r: np.ndarray, e: np.ndarray) -> Compressed:
    """One worker's compression + error feedback; `e` is updated in place."""
    c = cfg.c()
    slots = total_slots(cfg, tab)
    payload = np.zeros(payload_bytes(cfg, tab), np.uint8) if cfg.quant_bits in (1, 2, 3, 4) else None
    sel_idx = np.empty(max(slots, 1), np.int32)
    sel_val = np.empty(max(slots, 1), np.float32)
    sel_hat = np.empty(max(slots, 1), np.float32)
    stats = np.zeros((tab.n, 18), np.float32)
    lib().orc_compress(C.byref(c), tab.ref(), tab.n, _ptr(_chk(theta, np.float32)),
                       _ptr(_chk(theta_r, np.float32)), _ptr(_chk(e, np.float32)), _ptr(payload),
                       _ptr(sel_idx), _ptr(sel_val), _ptr(sel_hat), _ptr(stats))
    return Compressed(payload, sel_idx[:slots], sel_val[:slots], sel_hat[:slots], stats)


def bf16_round(x: float) -> float:
    """The bfloat16 nearest to x (ties to even), x an fp32 value; returned as a Python float."""
    return float(lib().orc_bf16_round(float(x)))


def bf16_round_d(x: float) -> float:
    """The bfloat16 nearest to the double x (ties to even), in one rounding."""
    return float(lib().orc_bf16_round_d(float(x)))


def decode_payload(cfg: Config, tab: Table, payload: np.ndarray):
    c = cfg.c()
    slots = total_slots(cfg, tab)
    idx = np.empty(max(slots, 1), np.int32)
    hat = np.empty(max(slots, 1), np.float32)
    lib().orc_decode_payload(C.byref(c), tab.ref(), tab.n, _ptr(_chk(payload, np.uint8)), _ptr(idx), _ptr(hat))
    return idx[:slots], hat[:slots]


def _ptr_array(arrs: Sequence[Optional[np.ndarray]]):
    pa = (C.c_void_p * len(arrs))()
    for i, a in enumerate(arrs):
        pa[i] = None if a is None else a.ctypes.data
    return pa


def aggregate_apply_sparse(cfg: Config, tab: Table, sel_idx: List[Optional[np.ndarray]],
                           sel_hat: List[Optional[np.ndarray]], theta: np.ndarray) -> None:
    c = cfg.c()
    assert len(sel_idx) == cfg.R and len(sel_hat) == cfg.R
    keep = [None if a is None else np.ascontiguousarray(a, np.int32) for a in sel_idx]
    keeph = [None if a is None else np.ascontiguousarray(a, np.float32) for a in sel_hat]
    lib().orc_aggregate_apply_sparse(C.byref(c), tab.ref(), tab.n, _ptr_array(keep),
                                     _ptr_array(keeph), _ptr(_chk(theta, np.float32)))


def aggregate_apply(cfg: Config, tab: Table, payloads: List[Optional[np.ndarray]], theta: np.ndarray) -> None:
    c = cfg.c()
    assert len(payloads) == cfg.R
    lib().orc_aggregate_apply(C.byref(c), tab.ref(), tab.n, _ptr_array(payloads),
                              _ptr(_chk(theta, np.float32)))


def outer_step(cfg: Config, tab: Table, theta: np.ndarray, theta_r: List[np.ndarray],
               e: List[np.ndarray]) -> List[np.ndarray]:
    """Full outer step; updates theta and every e in place, returns the R payloads."""
    c = cfg.c()
    nbytes = payload_bytes(cfg, tab)
    payloads = [np.zeros(nbytes, np.uint8) for _ in range(cfg.R)]
    for a in theta_r:
        _chk(a, np.float32)
    for a in e:
        _chk(a, np.float32)
    lib().orc_outer_step(C.byref(c), tab.ref(), tab.n, _ptr(_chk(theta, np.float32)),
                         _ptr_array(theta_r), _ptr_array(e), _ptr_array(payloads))
    return payloads


# ---------------------------------------------------------------- entropy-coded indices

def ixc_encode_chunk(idx: np.ndarray, L: int) -> tuple:
    """Golomb gap codes of one chunk's ascending indices: (bytes, number of bits)."""
    idx = _chk(idx, np.int32)
    pos = C.c_int64(0)
    lib().orc_ixc_encode_chunk(_ptr(idx), idx.size, L, None, C.byref(pos))
    nbits = pos.value
    out = np.zeros((nbits + 7) // 8 + 1, np.uint8)
    pos = C.c_int64(0)
    lib().orc_ixc_encode_chunk(_ptr(idx), idx.size, L, _ptr(out), C.byref(pos))
    return out, nbits


def ixc_decode_chunk(stream: np.ndarray, m_sel: int, L: int) -> tuple:
    stream = _chk(stream, np.uint8)
    idx = np.zeros(m_sel, np.int32)
    pos = C.c_int64(0)
    lib().orc_ixc_decode_chunk(_ptr(stream), C.byref(pos), m_sel, L, _ptr(idx))
    return idx, pos.value


def ixc_encode_payload(cfg: Config, tab: Table, payload: np.ndarray) -> np.ndarray:
    payload = _chk(payload, np.uint8)
    c = cfg.c()
    n = lib().orc_ixc_encode_payload(C.byref(c), tab.arr, tab.n, _ptr(payload), None)
    out = np.zeros(n, np.uint8)
    lib().orc_ixc_encode_payload(C.byref(c), tab.arr, tab.n, _ptr(payload), _ptr(out))
    return out


def ixc_decode_payload(cfg: Config, tab: Table, coded: np.ndarray) -> np.ndarray:
    coded = _chk(coded, np.uint8)
    c = cfg.c()
    out = np.zeros(payload_bytes(cfg, tab), np.uint8)
    lib().orc_ixc_decode_payload(C.byref(c), tab.arr, tab.n, _ptr(coded), _ptr(out))
    return out


# ---------------------------------------------------------------- dense baselines

def diloco_step(tab: Table, theta: np.ndarray, theta_r: List[np.ndarray], m: np.ndarray, beta_outer: float,
                alpha: float) -> None:
    """Eq. 1 in place on theta and the global momentum m (fp32 arrays)."""
    _chk(theta, np.float32); _chk(m, np.float32)
    arr = _ptr_array([_chk(a, np.float32) for a in theta_r])
    lib().orc_diloco_step(tab.arr, tab.n, len(theta_r), beta_outer, alpha, _ptr(theta), arr, _ptr(m))


def diloco_lom_step(tab: Table, theta: np.ndarray, theta_r: List[np.ndarray], m_r: List[np.ndarray],
                    beta_outer: float, alpha: float) -> None:
    """DiLoCo-LOM in place on theta and the per-replica momenta m_r (fp64 arrays)."""
    _chk(theta, np.float32)
    arr = _ptr_array([_chk(a, np.float32) for a in theta_r])
    marr = _ptr_array([_chk(a, np.float64) for a in m_r])
    lib().orc_diloco_lom_step(tab.arr, tab.n, len(theta_r), beta_outer, alpha, _ptr(theta), arr, marr)


# ---------------------------------------------------------------- Top-k / local-momentum variants (Alg. 2-4)

def lom_step(cfg: Config, tab: Table, theta: np.ndarray, theta_r: List[np.ndarray], m_r: List[np.ndarray],
             mu: float, sub_k: bool = False) -> None:
    """Alg. 2 (DiLoCo-LOM; with sub_k: DiLoCo-LOM-Sub-k) in place on theta and the fp32 momenta m_r."""
    c = cfg.c()
    lib().orc_lom_step(C.byref(c), tab.arr, tab.n, mu, int(sub_k), _ptr(_chk(theta, np.float32)),
                       _ptr_array([_chk(a, np.float32) for a in theta_r]),
                       _ptr_array([_chk(a, np.float32) for a in m_r]))


def diloco_topk_step(cfg: Config, tab: Table, theta: np.ndarray, theta_r: List[np.ndarray],
                     e: Optional[List[np.ndarray]], m: np.ndarray, mu: float) -> None:
    """Alg. 3 (DiLoCo + Top-k, error feedback when e is given) in place on theta, m and the e_r."""
    c = cfg.c()
    ea = _ptr_array([_chk(a, np.float32) for a in e]) if e is not None else None
    lib().orc_diloco_topk_step(C.byref(c), tab.arr, tab.n, mu, _ptr(_chk(theta, np.float32)),
                               _ptr_array([_chk(a, np.float32) for a in theta_r]), ea, _ptr(_chk(m, np.float32)))


def lom_topk_step(cfg: Config, tab: Table, theta: np.ndarray, theta_r: List[np.ndarray], m_r: List[np.ndarray],
                  e: Optional[List[np.ndarray]], mu: float) -> None:
    """Alg. 4 (DiLoCo-LOM + Top-k, error feedback when e is given) in place on theta, the m_r and the e_r."""
    c = cfg.c()
    ea = _ptr_array([_chk(a, np.float32) for a in e]) if e is not None else None
    lib().orc_lom_topk_step(C.byref(c), tab.arr, tab.n, mu, _ptr(_chk(theta, np.float32)),
                            _ptr_array([_chk(a, np.float32) for a in theta_r]),
                            _ptr_array([_chk(a, np.float32) for a in m_r]), ea)
