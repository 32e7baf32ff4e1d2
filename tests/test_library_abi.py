"""The C-ABI library builds, loads, and exports every symbol the header declares (no compute)."""
import ctypes
import os
import re

import torch

from paper_2607_23815_b200 import build, kvattn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "kvattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\([^;{}]*\)\s*;", text)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared_functions()
    assert {"kv_pool_create", "kv_append", "attn_extend", "attn_decode", "attn_mixed", "kv_evict", "kv_free",
            "kv_alloc"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in kvattn.h but not exported"
    # and the binding wraps each of them under the same name
    for n in names:
        assert n in kvattn._SIGNATURES, f"binding lacks {n}"


def test_host_only_calls():
    lib = kvattn.lib()
    assert lib.kv_status_str(0) == b"ok" and b"pages" in lib.kv_status_str(kvattn.KV_ERR_OOM)
    assert lib.kv_pool_destroy(None) == kvattn.KV_ERR_INVALID
    assert lib.kv_alloc(None, 1, None) == kvattn.KV_ERR_INVALID
    assert kvattn.kvattn_launch_count() >= 0
    h = ctypes.c_void_p()
    assert lib.kv_pool_create(8, 32, 2, 64, ctypes.byref(h)) == kvattn.KV_ERR_UNSUPPORTED      # page size
    if not torch.cuda.is_available():
        # without a device the library reports the failure instead of falling back to anything
        assert lib.kv_pool_create(8, 16, 2, 64, ctypes.byref(h)) == kvattn.KV_ERR_CUDA
        assert not h.value
