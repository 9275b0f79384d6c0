"""The C-ABI library loads and exports every symbol include/mtrains_b200.h declares; host-side
argument validation works without a GPU."""
import ctypes
import os
import re

import pytest

from paper_2305_01515_b200 import binding as mb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "mtrains_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mts_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 18
    lib = ctypes.CDLL(mb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(mb.EXPORTS) == names


def test_null_and_bad_arguments_are_rejected_on_the_host():
    L = mb.lib()
    assert L.mts_tables_create(None, None) == mb.ERR_INVALID_ARG
    assert b"null" in L.mts_last_error_string()
    h = ctypes.c_void_p()
    assert L.mts_cache_create(ctypes.byref(h), 4, 100, 16, 64, 1, 0, 0) == mb.ERR_INVALID_ARG   # ways != 32
    assert L.mts_cache_create(ctypes.byref(h), 0, 100, 32, 64, 1, 0, 0) == mb.ERR_INVALID_ARG   # no sets
    assert L.mts_cache_create(ctypes.byref(h), 4, 100, 32, 4, 1, 0, 0) == mb.ERR_ALIGNMENT      # 8-byte rows
    assert L.mts_tbe_forward(None, 1, None, None, 0, 0, None, None, 0, None, 0, None) == mb.ERR_INVALID_ARG
    assert L.mts_tbe_backward_workspace_bytes(None, 1, 10) == 0
    assert L.mts_cache_workspace_bytes(None, 10) == 0
    with pytest.raises(mb.MtsError):
        mb._check(mb.ERR_INVALID_ARG)


def test_table_description_is_validated_before_any_cuda_call():
    rows = (ctypes.c_int64 * 1)(10)
    dim = (ctypes.c_int32 * 1)(6)                    # 12-byte fp16 rows: not a 16-byte multiple
    woff = (ctypes.c_int64 * 1)(0)
    d = mb.TableDesc(1, mb.DTYPE_FP16, rows, dim, woff, ctypes.POINTER(ctypes.c_int32)(), 256, None, 256)
    h = ctypes.c_void_p()
    assert mb.lib().mts_tables_create(ctypes.byref(d), ctypes.byref(h)) == mb.ERR_ALIGNMENT
    rows[0] = 1 << 33
    dim[0] = 8
    assert mb.lib().mts_tables_create(ctypes.byref(d), ctypes.byref(h)) == mb.ERR_UNSUPPORTED
    rows[0] = 0
    assert mb.lib().mts_tables_create(ctypes.byref(d), ctypes.byref(h)) == mb.ERR_INVALID_ARG
