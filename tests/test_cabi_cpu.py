"""CPU-side checks of the C ABI: the library loads, exports every symbol the
header declares, and the calls that need no device behave."""
import ctypes as C
import os
import re

import pytest


@pytest.fixture(scope="module")
def xkv():
    from paper_2601_01204_b200 import build
    build.build()
    import paper_2601_01204_b200.xkv as m
    return m


def test_exports_match_header(xkv, repo_root):
    text = open(os.path.join(repo_root, "include", "xkv.h")).read()
    declared = re.findall(r"XKV_API\s+[\w\s\*]+?\b(\w+)\s*\(", text)
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(xkv.lib, name), name
    assert sorted(declared) == sorted(xkv.EXPORTED)


def test_workspace_bytes_and_param_validation(xkv):
    p = xkv.Params(budget=16384, max_frame_tokens=1374)
    nbytes = xkv.xkv_workspace_bytes(p)
    # two buffer sets of 4-bit K and V codes plus parameters (about 46 MiB) and the split-KV
    # partials of the attention kernel (about 34 MiB)
    assert 30 * 2 ** 20 < nbytes < 96 * 2 ** 20
    assert xkv.xkv_workspace_bytes(xkv.Params(head_dim=128)) == 0
    assert xkv.xkv_workspace_bytes(xkv.Params(kv_bits=3)) == 0
    assert xkv.xkv_workspace_bytes(xkv.Params(budget=0)) == 0
    h = C.c_void_p()
    bad = xkv.Params(head_dim=128)
    assert xkv.lib.xkv_create(C.byref(bad.c()), 256, 1 << 30, 0, C.byref(h)) == xkv.XKV_E_UNSUPPORTED
    bad = xkv.Params(kv_bits=2)
    assert xkv.lib.xkv_create(C.byref(bad.c()), 256, 1 << 30, 0, C.byref(h)) == xkv.XKV_E_UNSUPPORTED
    bad = xkv.Params(n_heads=0)
    assert xkv.lib.xkv_create(C.byref(bad.c()), 256, 1 << 30, 0, C.byref(h)) == xkv.XKV_E_INVALID
    good = xkv.Params()
    assert xkv.lib.xkv_create(C.byref(good.c()), 257, 1 << 30, 0, C.byref(h)) == xkv.XKV_E_INVALID  # misaligned
    assert xkv.lib.xkv_create(C.byref(good.c()), 256, 16, 0, C.byref(h)) == xkv.XKV_E_NOMEM
    assert xkv.lib.xkv_destroy(None) == xkv.XKV_E_INVALID
    assert xkv.lib.kv_quant_pack(None, None) == xkv.XKV_E_INVALID


def test_strerror(xkv):
    assert xkv.lib.xkv_strerror(0) == b"ok"
    for code in range(-8, 0):
        assert len(xkv.lib.xkv_strerror(code)) > 3
    assert b"unknown" in xkv.lib.xkv_strerror(-99)
