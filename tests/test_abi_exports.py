"""The C-ABI library loads without a GPU and exports every function include/rd.h declares; calls
that need no device return their documented error codes."""
import ctypes
import os
import re

import paper_2510_14961_b200 as rd
from paper_2510_14961_b200 import build as rd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "rd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    rd_build.build()
    names = _declared()
    assert "rd_df_step" in names and "rd_ar_step" in names and "rd_prefill" in names and "rd_load" in names
    L = rd.lib()
    missing = [n for n in names if not hasattr(L, n)]
    assert not missing, f"declared but not exported: {missing}"
    assert sorted(rd.EXPORTS) == names, "binding's export list and the header disagree"


def test_null_arguments_are_refused_without_a_device():
    L = rd.lib()
    assert L.rd_load(None, None, 0, 4, None) == rd.RD_E_INVALID_ARG
    assert L.rd_df_step(None, 4, 1, ctypes.c_float(0.0)) == rd.RD_E_INVALID_ARG
    assert L.rd_ar_step(None, 4) == rd.RD_E_INVALID_ARG
    assert L.rd_prefill(None, 0, None, 0, 0) == rd.RD_E_INVALID_ARG
    assert L.rd_sync(None) == rd.RD_E_INVALID_ARG
    assert L.rd_strerror(rd.RD_E_CAPACITY) == b"capacity exceeded (context or window)"
    assert L.rd_strerror(12345) == b"unknown error code"
