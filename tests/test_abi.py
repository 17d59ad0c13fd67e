"""The C-ABI library loads and exports every function that include/mate.h declares (no GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    with open(os.path.join(ROOT, "include", "mate.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mate_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2109_04312_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_three_calls():
    names = declared_functions()
    for need in ("mate_plan", "mate_attn_fwd", "mate_attn_bwd"):
        assert need in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_status_strings(lib):
    lib.mate_status_string.restype = ctypes.c_char_p
    seen = set()
    for s in range(0, -8, -1):
        msg = lib.mate_status_string(s).decode()
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 8
    assert lib.mate_status_string(-99).decode() == "unknown status"


def test_null_arguments_are_rejected_without_a_gpu(lib):
    # argument checks come before any CUDA call, so they work on a machine without a device
    out = ctypes.c_void_p()
    assert lib.mate_plan(None, None, 1, 8, 0, None, 1, 1, 1, None, ctypes.byref(out)) == -1
    assert lib.mate_plan_get(None, 0, None, None, None) == -1
    assert lib.mate_plan_useful_pairs(None, None) == -1
    assert lib.mate_plan_destroy(None) == 0
    f = ctypes.c_size_t()
    assert lib.mate_attn_workspace_bytes(None, 64, 0, 0, ctypes.byref(f), ctypes.byref(f)) == -1


def test_binding_fails_loudly_without_the_library(monkeypatch):
    from paper_2109_04312_b200 import api
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmate.so"))
    with pytest.raises(ImportError):
        api._load()
