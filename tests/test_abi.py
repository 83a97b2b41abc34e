"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import paper_2605_27003_b200 as pkg
from paper_2605_27003_b200 import build as pkg_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_symbols():
    text = open(os.path.join(ROOT, "include", "w4a4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(w4a4_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    pkg_build.build()
    lib = ctypes.CDLL(pkg.LIB_PATH)
    declared = _header_symbols()
    assert len(declared) >= 14
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(pkg.EXPORTED_SYMBOLS) == declared


def test_status_strings_and_tile_shape_without_a_device():
    pkg_build.build()
    assert pkg.w4a4_status_string(0) == "ok"
    assert "wait" in pkg.w4a4_status_string(6)
    bm, bn = pkg.w4a4_tile_shape()
    assert bm == 128 and bn % 64 == 0


def test_null_and_bad_arguments_are_rejected_without_a_device():
    pkg_build.build()
    lib = pkg.load_library()
    assert lib.w4a4_ctx_create(0, 128, 512, 16, None) == 1           # NULL out pointer
    out = ctypes.c_void_p()
    assert lib.w4a4_ctx_create(0, 0, 512, 16, ctypes.byref(out)) == 2   # max_M <= 0
    assert lib.w4a4_ctx_create(0, 128, 100, 16, ctypes.byref(out)) == 2  # K not a multiple of 64
    assert lib.w4a4_linear_forward(None, None, 1, 0, 0, None, None, None) == 1
    assert lib.w4a4_pack_weights(None, None, ctypes.byref(out)) == 1
    assert lib.w4a4_query_status(None) == 1
    assert lib.w4a4_debug_wait_probe(None, 1000, None) == 1
    assert lib.w4a4_debug_stalled_gemm(None, 1, 0, None, 0, 1000, None) == 1
    assert lib.w4a4_debug_set_tile_order(None, 2) == 1
    lib.w4a4_debug_fail_allocation_after(-1)                          # disarming needs no device
    lib.w4a4_destroy(None)
    lib.w4a4_ctx_destroy(None)
