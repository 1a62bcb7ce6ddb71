"""The C-ABI library builds, loads and exports every symbol include/gn.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gn_[A-Za-z0-9_]+)\s*\(", text)))


def test_header_declares_the_entry_points_of_the_path():
    names = declared_symbols()
    for must in ["gn_create", "gn_destroy", "gn_set_theta", "gn_set_subsample", "gn_fun", "gn_grad", "gn_Gv",
                 "gn_Gv_blockdiag", "gn_cg_solve"]:
        assert must in names


def test_library_exports_every_declared_symbol():
    import paper_1802_00130_b200 as gn
    handle = gn.lib()
    raw = ctypes.CDLL(gn.lib_path())
    for name in declared_symbols():
        assert hasattr(raw, name), f"{name} declared in gn.h but not exported"
    # and the binding knows each of them
    assert set(gn.exported_symbols()) == set(declared_symbols())
    assert handle is gn.lib()


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    import paper_1802_00130_b200 as gn
    handle = gn.lib()
    ctx = ctypes.c_void_p()
    widths = (ctypes.c_int32 * 2)(3, 2)
    dummy = ctypes.c_void_p(16)
    st = handle.gn_create(ctypes.byref(ctx), 1, widths, 1.0, 4, dummy, dummy, 1, None)
    assert st == 3 and not ctx.value          # GN_ECUDA, no context


def test_argument_errors_are_reported_before_any_launch():
    import paper_1802_00130_b200 as gn
    handle = gn.lib()
    ctx = ctypes.c_void_p()
    widths = (ctypes.c_int32 * 2)(3, 0)
    dummy = ctypes.c_void_p(16)
    assert handle.gn_create(ctypes.byref(ctx), 1, widths, 1.0, 4, dummy, dummy, 1, None) == 1   # width 0
    widths = (ctypes.c_int32 * 2)(3, 2)
    assert handle.gn_create(ctypes.byref(ctx), 1, widths, -1.0, 4, dummy, dummy, 1, None) == 1  # C <= 0
    assert handle.gn_create(ctypes.byref(ctx), 0, widths, 1.0, 4, dummy, dummy, 1, None) == 1   # L < 1
    assert handle.gn_create(ctypes.byref(ctx), 1, widths, 1.0, 4, None, dummy, 1, None) == 1    # NULL X
    assert handle.gn_num_params(None) == -1
    assert handle.gn_destroy(None) == 0
