"""Thin ctypes binding over libsparseloco's C ABI (see include/sparseloco.h).

Argument marshalling only: every step of the outer step runs in the CUDA kernels.  torch is
used for device memory and streams.  Importing this module loads the shared library and raises
if it is missing -- there is no CPU implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparseloco.so")

EXPORTS = (
    "sl_create", "sl_destroy", "sl_set_hyper", "sl_record_stride", "sl_payload_bytes", "sl_num_chunks",
    "sl_flat_elems", "sl_workspace_bytes", "sl_set_workspace", "sl_compress", "sl_aggregate_apply",
    "sl_outer_step", "sl_outer_step_host", "sl_validate_payload", "sl_read_stats", "sl_strerror",
    "sl_last_cuda_error", "sl_diloco_step", "sl_coded_payload_capacity", "sl_encode_payload", "sl_decode_payload", "sl_set_tile_copies", "sl_device_status", "sl_static_scratch_bytes", "sl_compress_tensor_static", "sl_set_ef_deferred", "sl_ef_pending", "sl_ef_flush", "sl_profile_enable", "sl_profile_read", "sl_profile_name", "sl_lom_step", "sl_diloco_topk_step", "sl_lom_topk_step", "sl_streaming_due",
    "sl_compress_bf16", "sl_aggregate_apply_bf16", "sl_outer_step_bf16", "sl_aggregate_apply_coded", "sl_ef_flush_bf16",
)
PROFILE_SLOTS = 9

SL_OK = 0
SL_ERR_INVALID_ARG, SL_ERR_ALIGNMENT, SL_ERR_UNSUPPORTED, SL_ERR_BAD_PAYLOAD = 1, 2, 3, 4
SL_ERR_CUDA, SL_ERR_NOMEM, SL_ERR_TOO_LARGE, SL_ERR_TIMEOUT = 5, 6, 7, 8


class SlError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(msg)
        self.status = status


class _TensorDesc(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("offset", C.c_int64)]


class _Config(C.Structure):
    _fields_ = [("chunk_elems", C.c_int32), ("tile_dim", C.c_int32), ("k", C.c_int32),
                ("R", C.c_int32), ("H", C.c_int32), ("beta", C.c_float), ("outer_lr", C.c_float),
                ("quant_bits", C.c_int32), ("ef_enabled", C.c_int32),
                ("divide_by_present", C.c_int32), ("bf16_storage", C.c_int32)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
            "(nvcc, sm_100a).  This package has no CPU fallback.")
    L = C.CDLL(LIB_PATH)
    P = C.c_void_p
    L.sl_create.argtypes = [P, P, C.c_int32, C.POINTER(P)]
    L.sl_destroy.argtypes = [P]
    L.sl_set_hyper.argtypes = [P, C.c_float, C.c_float, C.c_int32, C.c_int32]
    L.sl_record_stride.argtypes = [C.c_int32]
    L.sl_record_stride.restype = C.c_size_t
    L.sl_payload_bytes.argtypes = [P, C.POINTER(C.c_size_t)]
    L.sl_num_chunks.argtypes = [P, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.sl_flat_elems.argtypes = [P, C.POINTER(C.c_int64)]
    L.sl_workspace_bytes.argtypes = [P, C.POINTER(C.c_size_t)]
    L.sl_set_workspace.argtypes = [P, P, C.c_size_t]
    L.sl_compress.argtypes = [P, P, P, P, P, P]
    L.sl_aggregate_apply.argtypes = [P, P, P, P]
    L.sl_outer_step.argtypes = [P, P, P, P, P, P]
    L.sl_compress_bf16.argtypes = [P, P, P, P, P, P]
    L.sl_ef_flush_bf16.argtypes = [P, P, C.c_int32, P]
    L.sl_aggregate_apply_coded.argtypes = [P, P, P, P, P]
    L.sl_aggregate_apply_bf16.argtypes = [P, P, P, P]
    L.sl_outer_step_bf16.argtypes = [P, P, P, P, P, P]
    L.sl_outer_step_host.argtypes = [P, P, P, P, C.c_size_t, P, P, P, P]
    L.sl_profile_enable.argtypes = [P, C.c_int32]
    L.sl_profile_read.argtypes = [P, P, P]
    L.sl_profile_name.argtypes = [C.c_int32]
    L.sl_profile_name.restype = C.c_char_p
    L.sl_validate_payload.argtypes = [P, P, P, P]
    L.sl_diloco_step.argtypes = [P, P, P, P, C.c_float, P]
    L.sl_lom_step.argtypes = [P, P, P, P, C.c_float, C.c_int32, P]
    L.sl_diloco_topk_step.argtypes = [P, P, P, P, P, C.c_float, P]
    L.sl_lom_topk_step.argtypes = [P, P, P, P, P, C.c_float, P]
    L.sl_coded_payload_capacity.argtypes = [P, C.POINTER(C.c_size_t)]
    L.sl_encode_payload.argtypes = [P, P, P, P, P]
    L.sl_decode_payload.argtypes = [P, P, C.c_size_t, P, P]
    L.sl_set_tile_copies.argtypes = [P, C.c_int32]
    L.sl_device_status.argtypes = [P, P]
    L.sl_static_scratch_bytes.restype = C.c_size_t
    L.sl_compress_tensor_static.argtypes = [P, P, P, P, C.c_int64, C.c_int64, C.c_int32, C.c_float, P]
    L.sl_set_ef_deferred.argtypes = [P, C.c_int32]
    L.sl_ef_pending.argtypes = [P, C.POINTER(C.c_int32)]
    L.sl_ef_flush.argtypes = [P, P, C.c_int32, P]
    L.sl_read_stats.argtypes = [P, C.c_int32, P, P]
    L.sl_streaming_due.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.POINTER(C.c_int32)]
    L.sl_strerror.argtypes = [C.c_int]
    L.sl_strerror.restype = C.c_char_p
    L.sl_last_cuda_error.restype = C.c_char_p
    return L


_L = _load()


def _check(st: int) -> None:
    if st != SL_OK:
        msg = _L.sl_strerror(st).decode()
        if st == SL_ERR_CUDA:
            msg += ": " + _L.sl_last_cuda_error().decode()
        raise SlError(st, f"libsparseloco: {msg} (status {st})")


def _dev_ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _ptr_array(ptrs: Sequence[Optional[int]]):
    arr = (C.c_void_p * len(ptrs))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def record_stride(k: int) -> int:
    return _L.sl_record_stride(k)


def streaming_due(H: int, P: int, inner_step: int) -> int:
    """Fragment of Streaming SparseLoCo that synchronises after `inner_step` inner steps, or -1."""
    v = C.c_int32()
    _check(_L.sl_streaming_due(H, P, inner_step, C.byref(v)))
    return v.value


def static_scratch_bytes() -> int:
    return _L.sl_static_scratch_bytes()


def compress_tensor_static(theta_sync, theta_local, e, payload, rows: int, cols: int, k: int, beta: float) -> None:
    """sl_compress_tensor_static: one tensor of one worker, scratch inside the library, no allocation.
    Raises SlError (status SL_ERR_TOO_LARGE) when the tensor does not fit the fixed scratch."""
    _check(_L.sl_compress_tensor_static(_dev_ptr(theta_sync, torch.float32), _dev_ptr(theta_local, torch.float32),
                                        _dev_ptr(e, torch.float32), _dev_ptr(payload, torch.uint8), rows, cols, k,
                                        beta, _stream()))


class SparseLoCo:
    """One context = one tensor table + hyper-parameters on the current CUDA device.

    Method names mirror the C entry points: `compress`, `aggregate_apply`, `outer_step`,
    `outer_step_host`, `validate_payload`.  All work is enqueued on torch's current stream.
    """

    def __init__(self, shapes: Sequence[Sequence[int]], offsets: Optional[Sequence[int]] = None, *,
                 k: int, R: int, H: int = 1, beta: float = 0.95, outer_lr: float = 1.0,
                 ef_enabled: bool = True, divide_by_present: bool = False, chunk_elems: int = 4096,
                 tile_dim: int = 64, quant_bits: int = 2, alloc_workspace: bool = True,
                 bf16_storage: bool = False):
        n = len(shapes)
        descs = (_TensorDesc * n)()
        pos = 0
        for j, sh in enumerate(shapes):
            rows, cols = (1, sh[0]) if len(sh) == 1 else (sh[0], sh[1])
            off = offsets[j] if offsets is not None else (pos + 3) // 4 * 4
            descs[j] = _TensorDesc(rows, cols, off)
            pos = off + rows * cols
        cfg = _Config(chunk_elems, tile_dim, k, R, H, beta, outer_lr, quant_bits, int(ef_enabled),
                      int(divide_by_present), int(bf16_storage))
        # element type of theta, theta_local and e; the library has one set of entry points per type
        self.dtype = torch.bfloat16 if bf16_storage else torch.float32
        self._h = C.c_void_p()
        self.k, self.R = k, R
        self._beta, self._lr, self._ef, self._dbp = beta, outer_lr, int(ef_enabled), int(divide_by_present)
        _check(_L.sl_create(C.byref(cfg), descs, n, C.byref(self._h)))
        self.device = torch.device("cuda", torch.cuda.current_device())
        self._ws = None
        if alloc_workspace:
            self._ws = torch.empty(self.workspace_bytes(), dtype=torch.uint8, device=self.device)
            self.set_workspace(self._ws)

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            _L.sl_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- closed forms
    def payload_bytes(self) -> int:
        v = C.c_size_t()
        _check(_L.sl_payload_bytes(self._h, C.byref(v)))
        return v.value

    def num_chunks(self):
        a, b = C.c_int64(), C.c_int64()
        _check(_L.sl_num_chunks(self._h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def flat_elems(self) -> int:
        v = C.c_int64()
        _check(_L.sl_flat_elems(self._h, C.byref(v)))
        return v.value

    def workspace_bytes(self) -> int:
        v = C.c_size_t()
        _check(_L.sl_workspace_bytes(self._h, C.byref(v)))
        return v.value

    def set_workspace(self, ws: Optional[torch.Tensor]) -> None:
        self._ws = ws
        if ws is None:
            _check(_L.sl_set_workspace(self._h, None, 0))
        else:
            _check(_L.sl_set_workspace(self._h, _dev_ptr(ws), ws.numel() * ws.element_size()))

    def set_hyper(self, beta=None, outer_lr=None, ef_enabled=None, divide_by_present=None) -> None:
        if beta is not None:
            self._beta = beta
        if outer_lr is not None:
            self._lr = outer_lr
        if ef_enabled is not None:
            self._ef = int(ef_enabled)
        if divide_by_present is not None:
            self._dbp = int(divide_by_present)
        _check(_L.sl_set_hyper(self._h, self._beta, self._lr, self._ef, self._dbp))

    # -- the path
    def compress(self, theta_sync, theta_local, e, payload) -> None:
        fn = _L.sl_compress_bf16 if self.dtype == torch.bfloat16 else _L.sl_compress
        _check(fn(self._h, _dev_ptr(theta_sync, self.dtype), _dev_ptr(theta_local, self.dtype),
                  _dev_ptr(e, self.dtype), _dev_ptr(payload, torch.uint8), _stream()))

    def aggregate_apply(self, payloads: List[Optional[torch.Tensor]], theta_sync) -> None:
        arr = _ptr_array([_dev_ptr(p, torch.uint8) for p in payloads])
        fn = _L.sl_aggregate_apply_bf16 if self.dtype == torch.bfloat16 else _L.sl_aggregate_apply
        _check(fn(self._h, arr, _dev_ptr(theta_sync, self.dtype), _stream()))

    def outer_step(self, theta_sync, theta_local: List[torch.Tensor], e: Optional[List[torch.Tensor]],
                   payloads: List[torch.Tensor]) -> None:
        tl = _ptr_array([_dev_ptr(t, self.dtype) for t in theta_local])
        ea = _ptr_array([_dev_ptr(t, self.dtype) for t in e]) if e is not None else None
        pa = _ptr_array([_dev_ptr(t, torch.uint8) for t in payloads])
        fn = _L.sl_outer_step_bf16 if self.dtype == torch.bfloat16 else _L.sl_outer_step
        _check(fn(self._h, _dev_ptr(theta_sync, self.dtype), tl, ea, pa, _stream()))

    def outer_step_host(self, theta_sync, theta_local_host: List[torch.Tensor], dev_stage,
                        e: Optional[List[torch.Tensor]], payloads: List[torch.Tensor],
                        theta_sync_host: Optional[torch.Tensor] = None) -> None:
        for t in theta_local_host:
            assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
        tl = _ptr_array([t.data_ptr() for t in theta_local_host])
        ea = _ptr_array([_dev_ptr(t, torch.float32) for t in e]) if e is not None else None
        pa = _ptr_array([_dev_ptr(t, torch.uint8) for t in payloads])
        hp = None
        if theta_sync_host is not None:
            assert not theta_sync_host.is_cuda and theta_sync_host.is_contiguous()
            hp = theta_sync_host.data_ptr()
        _check(_L.sl_outer_step_host(self._h, _dev_ptr(theta_sync, torch.float32), tl,
                                     _dev_ptr(dev_stage, torch.float32), dev_stage.numel(), ea, pa, hp,
                                     _stream()))

    def diloco_step(self, theta_sync, theta_local: List[torch.Tensor], momentum, beta_outer: float) -> None:
        """Dense baseline (Eq. 1): theta_sync and momentum updated in place."""
        tl = _ptr_array([_dev_ptr(t, torch.float32) for t in theta_local])
        _check(_L.sl_diloco_step(self._h, _dev_ptr(theta_sync, torch.float32), tl, _dev_ptr(momentum, torch.float32),
                                 beta_outer, _stream()))

    # -- the paper's Top-k / local-momentum variants (Alg. 2-4 of its appendix), no quantiser
    def lom_step(self, theta_sync, theta_local: List[torch.Tensor], m_r: List[torch.Tensor], mu: float,
                 sub_k: bool = False) -> None:
        tl = _ptr_array([_dev_ptr(t, torch.float32) for t in theta_local])
        ma = _ptr_array([_dev_ptr(t, torch.float32) for t in m_r])
        _check(_L.sl_lom_step(self._h, _dev_ptr(theta_sync, torch.float32), tl, ma, mu, int(sub_k), _stream()))

    def diloco_topk_step(self, theta_sync, theta_local: List[torch.Tensor], e: Optional[List[torch.Tensor]],
                         momentum, mu: float) -> None:
        tl = _ptr_array([_dev_ptr(t, torch.float32) for t in theta_local])
        ea = _ptr_array([_dev_ptr(t, torch.float32) for t in e]) if e is not None else None
        _check(_L.sl_diloco_topk_step(self._h, _dev_ptr(theta_sync, torch.float32), tl, ea,
                                      _dev_ptr(momentum, torch.float32), mu, _stream()))

    def lom_topk_step(self, theta_sync, theta_local: List[torch.Tensor], m_r: List[torch.Tensor],
                      e: Optional[List[torch.Tensor]], mu: float) -> None:
        """theta_local is consumed: on return buffer r holds worker r's Nesterov direction."""
        tl = _ptr_array([_dev_ptr(t, torch.float32) for t in theta_local])
        ma = _ptr_array([_dev_ptr(t, torch.float32) for t in m_r])
        ea = _ptr_array([_dev_ptr(t, torch.float32) for t in e]) if e is not None else None
        _check(_L.sl_lom_topk_step(self._h, _dev_ptr(theta_sync, torch.float32), tl, ma, ea, mu, _stream()))

    def coded_payload_capacity(self) -> int:
        v = C.c_size_t()
        _check(_L.sl_coded_payload_capacity(self._h, C.byref(v)))
        return v.value

    def encode_payload(self, payload, coded, coded_bytes: torch.Tensor) -> None:
        """12-bit payload -> entropy-coded payload; the size lands in `coded_bytes` (device int64[1])."""
        assert coded_bytes.dtype == torch.int64 and coded_bytes.numel() == 1
        _check(_L.sl_encode_payload(self._h, _dev_ptr(payload, torch.uint8), _dev_ptr(coded, torch.uint8),
                                    _dev_ptr(coded_bytes), _stream()))

    def decode_payload(self, coded, payload, coded_bytes: int = 0) -> None:
        """Entropy-coded payload -> 12-bit payload.  `coded_bytes` = readable bytes of `coded`
        (0: the tensor's size); a damaged input shows in device_status() as SL_ERR_BAD_PAYLOAD."""
        _check(_L.sl_decode_payload(self._h, _dev_ptr(coded, torch.uint8), coded_bytes or coded.numel(),
                                    _dev_ptr(payload, torch.uint8), _stream()))

    def aggregate_apply_coded(self, coded: List[Optional[torch.Tensor]], theta_sync,
                              coded_bytes: Optional[Sequence[int]] = None) -> None:
        """Decode, average and apply straight from entropy-coded payloads (None = absent worker).
        `coded_bytes[r]` = readable bytes of coded[r] (default: the tensor's size)."""
        arr = _ptr_array([_dev_ptr(p, torch.uint8) for p in coded])
        sizes = (C.c_size_t * len(coded))()
        for r, p in enumerate(coded):
            sizes[r] = 0 if p is None else int(coded_bytes[r] if coded_bytes is not None and coded_bytes[r] else p.numel())
        _check(_L.sl_aggregate_apply_coded(self._h, arr, sizes, _dev_ptr(theta_sync, self.dtype), _stream()))

    def set_tile_copies(self, use_tensor_maps: bool) -> None:
        _check(_L.sl_set_tile_copies(self._h, int(use_tensor_maps)))

    def device_status(self) -> int:
        """Synchronises the current stream; returns (and clears) the status the kernels recorded."""
        return int(_L.sl_device_status(self._h, _stream()))

    def set_ef_deferred(self, on: bool = True) -> None:
        _check(_L.sl_set_ef_deferred(self._h, int(on)))

    def ef_pending(self) -> bool:
        v = C.c_int32()
        _check(_L.sl_ef_pending(self._h, C.byref(v)))
        return bool(v.value)

    def ef_flush(self, e: Optional[List[torch.Tensor]] = None, keep_pending: bool = False) -> None:
        ea = _ptr_array([_dev_ptr(t, self.dtype) if t is not None else None for t in e]) if e is not None else None
        fn = _L.sl_ef_flush_bf16 if self.dtype == torch.bfloat16 else _L.sl_ef_flush
        _check(fn(self._h, ea, int(keep_pending), _stream()))

    def profile_enable(self, on: bool = True) -> None:
        _check(_L.sl_profile_enable(self._h, int(on)))

    def profile_read(self):
        """{kernel name: (total ms, launches)} since the last read; waits for the recorded events."""
        ms = (C.c_float * PROFILE_SLOTS)()
        n = (C.c_int64 * PROFILE_SLOTS)()
        _check(_L.sl_profile_read(self._h, ms, n))
        return {_L.sl_profile_name(i).decode(): (ms[i], n[i]) for i in range(PROFILE_SLOTS)}

    def validate_payload(self, payload, status: torch.Tensor) -> None:
        assert status.dtype == torch.int32
        _check(_L.sl_validate_payload(self._h, _dev_ptr(payload, torch.uint8), _dev_ptr(status), _stream()))

    def read_stats(self, worker: int, n_tensors: int) -> torch.Tensor:
        out = torch.empty(n_tensors * 8, dtype=torch.float32, device=self.device)
        _check(_L.sl_read_stats(self._h, worker, _dev_ptr(out), _stream()))
        return out.view(n_tensors, 8)
