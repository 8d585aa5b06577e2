"""Host-only checks of the C-ABI library: it loads, exports every function the header
declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2604_06746_b200 import build
    build.build()
    from paper_2604_06746_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "structkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(structkv_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_exported(B):
    names = declared_functions()
    assert {"structkv_score_layer", "structkv_pivot", "structkv_select", "structkv_compact"} <= set(names)
    for name in names:
        assert hasattr(B.lib, name), name


def test_version_and_status_strings(B):
    assert B.version() >= 100
    seen = {B.lib.structkv_status_string(s) for s in range(6)}
    assert len(seen) == 6 and all(seen)
    assert B.lib.structkv_status_string(99)


def test_workspace_bytes(B):
    good = B.Config(32, 8, 128, 64, 131072, B.BF16)
    n = B.workspace_bytes(good)
    assert n > 0 and n % 256 == 0
    assert B.workspace_bytes(B.Config(32, 8, 128, 64, 262144, B.BF16)) > n
    for bad in (B.Config(32, 5, 128, 64, 4096, B.BF16),     # heads not a multiple of KV heads
                B.Config(32, 8, 96, 64, 4096, B.BF16),      # unsupported head_dim
                B.Config(32, 8, 128, 0, 4096, B.BF16),      # empty window
                B.Config(32, 8, 128, 64, 32, B.BF16),       # max_seq below the window
                B.Config(32, 8, 128, 64, 4096, 7)):         # unknown dtype
        assert B.workspace_bytes(bad) == 0


def test_create_rejects_bad_arguments_on_the_host(B):
    h = ctypes.c_void_p()
    cfg = B.Config(8, 2, 64, 32, 2048, B.FP32)
    assert B.lib.structkv_create(None, ctypes.byref(cfg), None, 0) == B.ERR_INVALID_ARG
    assert B.lib.structkv_create(ctypes.byref(h), None, None, 0) == B.ERR_INVALID_ARG
    assert B.lib.structkv_create(ctypes.byref(h), ctypes.byref(cfg), None, 0) == B.ERR_WORKSPACE
    assert B.lib.structkv_create(ctypes.byref(h), ctypes.byref(cfg), 256, 16) == B.ERR_WORKSPACE
    bad = B.Config(8, 2, 80, 32, 2048, B.FP32)
    assert B.lib.structkv_create(ctypes.byref(h), ctypes.byref(bad), None, 0) == B.ERR_UNSUPPORTED
    assert not h.value
    # every entry point refuses a null context without dereferencing anything
    assert B.lib.structkv_score_layer(None, None, None, 0, 0, 0, 1.0, 1.0, None, None, None, None, 0, None) == B.ERR_INVALID_ARG
    assert B.lib.structkv_pivot(None, None, 0, None, -1, None, None, None) == B.ERR_INVALID_ARG
    assert B.lib.structkv_accumulate(None, None, 0, 0, 0, 1.0, None, None) == B.ERR_INVALID_ARG
    assert B.lib.structkv_select(None, None, 0, 0, 0, 0, 0, None, None) == B.ERR_INVALID_ARG
    assert B.lib.structkv_compact(None, None, 0, 0, 0, 0, 0, None, 0, None, None) == B.ERR_INVALID_ARG
    assert B.lib.structkv_poll_device_status(None, None) == B.ERR_INVALID_ARG
    B.lib.structkv_destroy(None)
