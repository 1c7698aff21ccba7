"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed),
and argument validation that happens before any device work returns the documented status."""
import ctypes
import os
import re

import pytest

from paper_2411_17178_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_exports_match_header(lib):
    text = open(os.path.join(ROOT, "include", "litevar.h")).read()
    declared = set(re.findall(r"\b(litevar_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    seen = set()
    for code in range(8):
        s = lib.litevar_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert lib.litevar_status_string(99).decode() == "unknown status"


def test_plan_argument_validation_before_device_work(lib):
    scales = (ctypes.c_int32 * 4)(1, 2, 3, 4)
    win = binding._Window()
    win.shape, win.n_global_scales, win.rho_num, win.rho_den, win.n_sets = 0, 3, 1, 4, 1
    out = ctypes.c_void_p()
    INV, UNS = 1, 2

    def call(sc=scales, n=4, heads=2, hd=64, w=win):
        return lib.litevar_attn_plan(sc, n, heads, hd, 0.0, ctypes.byref(w) if w is not None else None, None,
                                     None, ctypes.byref(out))

    assert call(sc=None) == INV
    assert call(w=None) == INV
    assert call(n=0) == INV
    assert call(n=17) == INV
    assert call(heads=0) == INV
    assert call(hd=32) == UNS
    bad = (ctypes.c_int32 * 4)(1, 0, 3, 4)
    assert call(sc=bad) == INV
    bad = (ctypes.c_int32 * 4)(1, 2, 3, 257)
    assert call(sc=bad) == INV
    w2 = binding._Window()
    w2.shape, w2.n_global_scales, w2.rho_num, w2.rho_den, w2.n_sets = 0, 3, 1, 0, 1
    assert call(w=w2) == INV
    w3 = binding._Window()
    w3.shape, w3.n_global_scales, w3.rho_num, w3.rho_den, w3.n_sets = 7, 3, 1, 4, 1
    assert call(w=w3) == INV
    assert out.value is None
    assert lib.litevar_attn_plan(scales, 4, 2, 64, 0.0, ctypes.byref(win), None, None, None) == INV


def test_null_plan_calls(lib):
    assert lib.litevar_plan_poll_device_status(None) == 1
    assert lib.litevar_plan_set_kernel(None, 0) == 1
    assert lib.litevar_plan_step_kernel(None, 1, 1, None) == 1
    assert lib.litevar_plan_stats(None, 1, 0, None, None, None, None) == 1
    lib.litevar_plan_destroy(None)
