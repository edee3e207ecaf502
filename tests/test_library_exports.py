"""CPU-side checks of the boundary: the shared library loads, exports every symbol the header
declares, and its host-only closed forms agree with the oracle's.  No device work."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sparseloco.h")


def declared_symbols():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(sl_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as g
    g.build()
    from paper_2508_15706_b200 import binding as B
    lib = C.CDLL(B.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 15
    for nm in names:
        assert hasattr(lib, nm), f"{nm} declared in sparseloco.h but not exported"
    assert set(names) == set(B.EXPORTS)


def test_record_stride_matches_oracle():
    import oracle as O
    from paper_2508_15706_b200 import binding as B
    for k in range(1, 257):
        assert B.record_stride(k) == O.record_stride(k)


def test_error_strings():
    from paper_2508_15706_b200 import binding as B
    lib = C.CDLL(B.LIB_PATH)
    lib.sl_strerror.restype = C.c_char_p
    seen = {lib.sl_strerror(i) for i in range(8)}
    assert len(seen) == 8 and b"ok" in seen


def test_null_arguments_are_rejected_without_a_device():
    from paper_2508_15706_b200 import binding as B
    lib = C.CDLL(B.LIB_PATH)
    assert lib.sl_create(None, None, 0, None) == B.SL_ERR_INVALID_ARG
    assert lib.sl_destroy(None) == B.SL_ERR_INVALID_ARG
    assert lib.sl_compress(None, None, None, None, None, None) == B.SL_ERR_INVALID_ARG
    assert lib.sl_outer_step(None, None, None, None, None, None) == B.SL_ERR_INVALID_ARG
    assert lib.sl_aggregate_apply(None, None, None, None) == B.SL_ERR_INVALID_ARG


def test_create_rejects_bad_tensor_tables_on_the_host():
    """Checked before any device call: overlapping element ranges (chunks of two tensors would race),
    sizes that overflow the 64-bit element arithmetic, a column count beyond 32 bits."""
    from paper_2508_15706_b200 import binding as B
    lib = C.CDLL(B.LIB_PATH)
    cfg = B._Config(4096, 64, 64, 2, 1, 0.9, 1.0, 2, 1, 0)

    def create(descs):
        arr = (B._TensorDesc * len(descs))(*[B._TensorDesc(r, c, o) for (r, c, o) in descs])
        out = C.c_void_p()
        st = lib.sl_create(C.byref(cfg), arr, len(descs), C.byref(out))
        assert out.value is None
        return st

    assert create([(64, 64, 0), (64, 64, 4092)]) == B.SL_ERR_INVALID_ARG          # second starts inside the first
    assert create([(1, 100, 4096), (64, 64, 0), (1, 8, 4100)]) == B.SL_ERR_INVALID_ARG  # unordered table, still found
    assert create([(1 << 41, 1 << 30, 0)]) == B.SL_ERR_TOO_LARGE                   # rows * cols overflows
    assert create([(1, 1 << 31, 0)]) == B.SL_ERR_TOO_LARGE                         # cols beyond 32 bits
    assert create([(64, 64, -4)]) == B.SL_ERR_INVALID_ARG
