"""The C-ABI library loads on a machine without a GPU and exports every function that
include/ef21.h declares; argument errors are reported without touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2106_05203_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ef21.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ef21_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = declared_functions()
    for must in ("ef21_create", "ef21_load_shards", "ef21_init", "ef21_step", "ef21_topk"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_signatures_cover_the_header():
    import importlib.util
    spec = importlib.util.find_spec("paper_2106_05203_b200.binding")
    src = open(spec.origin).read()
    for name in declared_functions():
        assert f'"{name}"' in src, f"binding.py has no signature for {name}"


def test_host_side_argument_checks(lib):
    lib.ef21_workspace_bytes.restype = ctypes.c_size_t
    lib.ef21_workspace_bytes.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64]
    assert lib.ef21_workspace_bytes(20, 112, 1, 8124) > 8124 * 112 * 4
    assert lib.ef21_workspace_bytes(0, 112, 1, 8124) == 0        # n < 1
    assert lib.ef21_workspace_bytes(20, 112, 113, 8124) == 0     # k > d
    assert lib.ef21_workspace_bytes(20, 112, 0, 8124) == 0       # k < 1
    assert lib.ef21_workspace_bytes(20, 1 << 31, 1, 0) == 0      # d too large for int32 indices
    assert lib.ef21_workspace_bytes(20, 112, 1, -1) == 0
    lib.ef21_topk_workspace_bytes.restype = ctypes.c_size_t
    lib.ef21_topk_workspace_bytes.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int32]
    assert lib.ef21_topk_workspace_bytes(64, 1 << 22, 4194) > 0
    assert lib.ef21_topk_workspace_bytes(0, 10, 1) == 0
    lib.ef21_status_string.restype = ctypes.c_char_p
    assert lib.ef21_status_string(0) == b"ok"
    assert b"wait" in lib.ef21_status_string(5)
    # create rejects bad scalars / null workspace before any CUDA call
    lib.ef21_create.restype = ctypes.c_int
    lib.ef21_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int32, ctypes.c_int64, ctypes.c_int32,
                                ctypes.c_float, ctypes.c_float, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t,
                                ctypes.c_void_p]
    h = ctypes.c_void_p()
    assert lib.ef21_create(ctypes.byref(h), 4, 64, 4, 0.1, 0.1, 200, None, 1 << 30, None) == 1
    assert lib.ef21_create(ctypes.byref(h), 4, 64, 4, -0.1, 0.1, 200, ctypes.c_void_p(256), 1 << 30, None) == 1
    assert lib.ef21_create(ctypes.byref(h), 4, 64, 4, float("nan"), 0.1, 200, ctypes.c_void_p(256), 1 << 30, None) == 1
    assert lib.ef21_create(ctypes.byref(h), 4, 64, 4, 0.1, 0.1, 200, ctypes.c_void_p(256), 16, None) == 3
    assert lib.ef21_create(ctypes.byref(h), 4, 64, 4, 0.1, 0.1, 200, ctypes.c_void_p(260), 1 << 30, None) == 3
    assert h.value is None
    lib.ef21_destroy.argtypes = [ctypes.c_void_p]
    lib.ef21_destroy(None)
