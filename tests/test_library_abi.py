"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every function
include/twa.h declares (no compute is launched here)."""

import ctypes
import os
import re

from paper_2205_13104_b200 import twa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "twa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(twa_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_header_and_binding_list_the_same_entry_points():
    assert _declared_functions() == sorted(twa.EXPORTS)


def test_library_builds_loads_and_exports_every_symbol():
    twa.build_library()
    lib = ctypes.CDLL(twa.LIB_PATH)
    for name in _declared_functions():
        assert hasattr(lib, name), name
    for name in twa.EXPORTS:
        assert callable(getattr(twa, name)), name


def test_host_only_queries():
    twa.build_library()
    assert twa.twa_basis_col_stride(1000, 8) == 1024
    assert twa.twa_basis_col_stride(1001, 4) == 512          # 501 bytes -> 512
    assert twa.twa_basis_col_stride(7, 32) == 128
    assert twa.twa_basis_bytes(1000, 3, 8) == 3 * 1024
    assert twa.twa_workspace_bytes(10, 2, 8) > 0
    assert twa.twa_strerror(0) == "ok"
    assert "aligned" in twa.twa_strerror(twa.TWA_ERR_MISALIGNED)
