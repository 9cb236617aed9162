"""The C-ABI library loads, exports every symbol the header declares, and its host-side
argument validation works without a GPU (no compute call is made here)."""
import ctypes as C
import os
import re

import pytest

from paper_2608_26140_b200 import binding as ab
from paper_2608_26140_b200 import build as abuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    abuild.build()
    return ab.load_library()


def header_functions():
    src = open(os.path.join(ROOT, "include", "acache.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(acache_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = header_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ab.EXPORTS) == names


def desc(**kw):
    d = dict(hidden=256, n_heads=4, n_kv_heads=4, head_dim=64, ffn=1024, rms_eps=1e-5, qkv_bias=0,
             max_batch=2, max_ctx=256, max_affix=128, max_rows=64, max_masked=32, max_vocab=0, max_block=0)
    d.update(kw)
    return ab.ModelDesc(*[d[f] for f, _ in ab.ModelDesc._fields_])


def test_create_validates_shapes(lib):
    h = C.c_void_p()
    assert lib.acache_create(C.byref(desc()), C.byref(h)) == ab.OK and h.value
    assert lib.acache_workspace_bytes(h) > 0
    assert lib.acache_launch_count(h) == 0
    lib.acache_destroy(h)
    for bad, code in [(dict(head_dim=96), ab.ERR_UNSUPPORTED_SHAPE), (dict(n_kv_heads=3), ab.ERR_UNSUPPORTED_SHAPE),
                      (dict(ffn=1000), ab.ERR_UNSUPPORTED_SHAPE), (dict(hidden=0), ab.ERR_INVALID_ARG),
                      (dict(max_batch=0), ab.ERR_INVALID_ARG), (dict(hidden=192), ab.ERR_UNSUPPORTED_SHAPE)]:
        h = C.c_void_p()
        assert lib.acache_create(C.byref(desc(**bad)), C.byref(h)) == code, bad
        assert not h.value
    assert lib.acache_create(None, C.byref(h)) == ab.ERR_INVALID_ARG


def test_workspace_grows_with_problem_size(lib):
    h1, h2 = C.c_void_p(), C.c_void_p()
    lib.acache_create(C.byref(desc()), C.byref(h1))
    lib.acache_create(C.byref(desc(max_rows=128, max_batch=4)), C.byref(h2))
    assert lib.acache_workspace_bytes(h2) > lib.acache_workspace_bytes(h1)
    lib.acache_destroy(h1)
    lib.acache_destroy(h2)


def test_calls_without_workspace_are_rejected_before_any_launch(lib):
    h = C.c_void_p()
    lib.acache_create(C.byref(desc()), C.byref(h))
    req = ab.Request(1, 256, 0, 128, None, 0, None, 0, None, None, None, 0)
    kv = ab.KV(None, None, 0, 256)
    st = lib.acache_score_anchors(h, C.byref(req), None, C.byref(kv), None, 0, 0, None)
    assert st == ab.ERR_WORKSPACE
    assert b"workspace" in lib.acache_last_error(h)
    assert lib.acache_select_topk(h, None, 1, 10, 11, None, None) == ab.ERR_INVALID_ARG
    assert lib.acache_select_topk(h, None, 1, 10, 0, None, None) == ab.OK        # K = 0: nothing to do
    assert lib.acache_set_workspace(h, None, 1 << 30, None) == ab.ERR_INVALID_ARG
    assert lib.acache_set_workspace(h, 256, 16, None) == ab.ERR_WORKSPACE
    assert lib.acache_launch_count(h) == 0
    lib.acache_destroy(h)


def test_k_from_ratio_host_function(lib):
    f = lib.acache_k_from_ratio
    assert [f(512, 0.2), f(2048, 0.2), f(1024, 0.2), f(128, 0.2)] == [103, 410, 205, 26]
    assert f(10, 0.3) == 3 and f(100, 0.0) == 0 and f(100, 1.0) == 100 and f(100, 2.0) == 100
    assert f(100, 1e-4) == 1 and f(0, 0.5) == 0 and f(100, -1.0) == 0
    from oracle import acache_oracle as orc
    for L in (1, 7, 100, 512, 8192):
        for r in (0.0, 0.05, 0.1, 0.2, 0.35, 0.5, 1.0):
            assert f(L, r) == orc.k_from_ratio(L, r)
