"""CPU-side checks of the boundary: the library builds, loads and exports every symbol that
include/dyspec.h declares; host-only entry points behave; nothing here launches a kernel."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding as B
    return B


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "dyspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dyspec_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_expected_calls():
    names = _declared_functions()
    for must in ("dyspec_build_tree_mask", "dyspec_tree_attention", "dyspec_tree_attention_ragged",
                 "dyspec_plan_create", "dyspec_plan_destroy", "dyspec_plan_workspace_bytes"):
        assert must in names


def test_library_exports_every_declared_symbol(binding):
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in _declared_functions():
        assert hasattr(lib, name), f"{name} declared in dyspec.h but not exported"
        assert name in binding.SIGNATURES, f"{name} has no binding signature"
        assert hasattr(binding, name), f"binding has no wrapper named {name}"


def test_host_only_entry_points(binding):
    B = binding
    assert B.dyspec_version() >= 100
    assert B.dyspec_words_per_row(0) == 4
    assert B.dyspec_words_per_row(1) == 4
    assert B.dyspec_words_per_row(128) == 4
    assert B.dyspec_words_per_row(129) == 8
    assert B.dyspec_words_per_row(768) == 24
    assert B.dyspec_words_per_row(1024) == 32
    assert B.dyspec_words_per_row(2048) == 64
    assert B.dyspec_words_per_row(2049) < 0
    assert B.dyspec_error_string(0) == "ok"
    for code in range(-6, 0):
        assert B.dyspec_error_string(code) not in ("ok", "unknown error code")
    assert B.dyspec_error_string(-99) == "unknown error code"


def test_argument_errors_are_reported_before_any_launch(binding):
    B = binding
    lib = B.lib
    # mask builder: bad sizes are rejected on the host (no device pointer is touched)
    assert lib.dyspec_build_tree_mask(None, -1, None, None, 4, None, None) == -1
    assert lib.dyspec_build_tree_mask(None, 5, None, None, 3, None, None) == -1          # W not a multiple of 4
    assert lib.dyspec_build_tree_mask(None, 3000, None, None, 96, None, None) == -2       # > DYSPEC_MAX_NODES
    assert lib.dyspec_build_tree_mask(None, 200, None, None, 4, None, None) == -1         # 32*W < n
    assert lib.dyspec_build_tree_mask(None, 0, None, None, 4, None, None) == 0            # empty tree: no-op
    assert lib.dyspec_build_tree_mask(None, 5, None, None, 4, None, None) == -1           # NULL pointers
    # plan: unsupported shapes
    h = ctypes.c_void_p()
    i32 = (ctypes.c_int32 * 1)
    i64 = (ctypes.c_int64 * 1)
    def create(hq, hkv, d, L=16, n=4, W=4, total=None, off=0):
        total = L + n if total is None else total
        return lib.dyspec_plan_create(ctypes.byref(h), hq, hkv, d, 1, ctypes.cast(i32(L), ctypes.c_void_p),
                                      ctypes.cast(i32(n), ctypes.c_void_p), ctypes.cast(i64(off), ctypes.c_void_p),
                                      total, W, 0.0)
    assert create(6, 4, 64) == -2            # H_q not a multiple of H_kv
    assert create(48, 4, 64) == -2           # g = 12
    assert create(4, 4, 96) == -2            # head_dim
    assert create(4, 4, 64, W=6) == -1
    assert create(4, 4, 64, n=2049, W=68) == -2
    assert create(4, 4, 64, n=200, W=4) == -1
    assert create(4, 4, 64, total=10) == -1  # request does not fit in the cache
    assert create(0, 4, 64) == -1
    assert lib.dyspec_tree_attention_ragged(None, None, None, None, None, None, None, 0, None, None) == -1
    assert lib.dyspec_set_default_shape(4, 4, 96, 4, 0.0) == -2
    assert lib.dyspec_set_tuning(7, 0, 1) == -1
    assert lib.dyspec_plan_destroy(None) == 0
