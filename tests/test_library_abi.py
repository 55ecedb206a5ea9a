"""The C-ABI library builds without a GPU, loads, and exports every symbol the header declares (no compute calls)."""
import ctypes
import os
import re

from paper_2402_14160_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    header = open(os.path.join(ROOT, "include", "rsd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rsd_[a-z0-9_]+)\s*\(", header))
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.rsd_rng_layout() == 3
    lib.rsd_sbs_workspace_bytes.restype = ctypes.c_size_t
    assert lib.rsd_sbs_workspace_bytes(4, 8, 8) >= 4 * 8 * 8 * 8 + 4 * 8 * 4
    lib.rsd_sbs_tree_workspace_bytes.restype = ctypes.c_size_t
    assert lib.rsd_sbs_tree_workspace_bytes(4, 8, 8) >= 4 * 57 * 8 * 12 + 4 * 57 * 8


def test_argument_validation_needs_no_gpu():
    lib = api.lib()
    rows = api.RsdRows(None, 0, 0, 0, 0)
    k = (ctypes.c_int32 * 1)(1)
    code = lib.rsd_gumbel_topk_draft(ctypes.byref(rows), 1, 1, 8, k, k, 1, 0, 0, 0, None, None, None, None, None, 0, None, None)
    assert code == 1 and b"null" in lib.rsd_last_error()
    rows = api.RsdRows(16, 7, 0, 8, 8)
    code = lib.rsd_gumbel_topk_draft(ctypes.byref(rows), 1, 1, 8, k, k, 1, 0, 0, 0, None, None, None, None, None, 0, None, None)
    assert code == 2 and b"dtype" in lib.rsd_last_error()
    rows = api.RsdRows(16, 0, 0, 8, 8)
    code = lib.rsd_gumbel_topk_draft(ctypes.byref(rows), 1, 1, 0, k, k, 1, 0, 0, 0, None, None, None, None, None, 0, None, None)
    assert code == 2
