"""The C-ABI library loads on a machine without a GPU and exports every symbol
that include/dk.h declares (no compute call is made here)."""
import ctypes
import os
import re

from paper_2207_00083_b200 import binding as dk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dk.h")).read()
    return sorted(set(re.findall(r"DK_API\s+[\w\s\*]+?\b(dk_\w+)\s*\(", text)))


def test_header_declares_the_path_entry_points():
    syms = declared_symbols()
    for name in ("dk_encode", "dk_linear_fwd", "dk_decode_verify", "dk_masked_linear", "dk_linear_bwd_wgrad"):
        assert name in syms


def test_library_exports_every_declared_symbol():
    L = dk.lib()
    for name in declared_symbols():
        assert hasattr(L, name), name
    assert sorted(dk.EXPORTS) == declared_symbols()


def test_struct_layouts_match_header():
    assert ctypes.sizeof(dk.dk_problem) == 14 * 4
    assert ctypes.sizeof(dk.dk_verdict) == 24
    assert dk.dk_verdict.first_index.offset == 8
    assert ctypes.sizeof(dk.dk_fault) == 24


def test_host_side_argument_checks_need_no_gpu():
    L = dk.lib()
    n = ctypes.c_size_t()
    p = dk.dk_problem(dk.DK_CONV2D, dk.DK_NHWC, 64, 64, 32, 32, 3, 3, 1, 1, 4, 32, 0, 0.0)
    assert L.dk_workspace_bytes(ctypes.byref(p), ctypes.byref(n)) == 0
    e = 6 * 32
    assert n.value >= 4 * (e * 64 * 32 * 32 * 2)
    bad = dk.dk_problem(dk.DK_CONV2D, dk.DK_NHWC, 64, 64, 32, 32, 3, 3, 1, 1, 9, 32, 0, 0.0)
    assert L.dk_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == 2      # DK_ERR_SHAPE
    bad = dk.dk_problem(7, dk.DK_NHWC, 64, 64, 32, 32, 3, 3, 1, 1, 4, 32, 0, 0.0)
    assert L.dk_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == 1      # DK_ERR_INVALID_ARG
    assert L.dk_status_string(3) == b"DK_ERR_SINGULAR"
