"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2604_12056_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_12056_b200 import build
    build.build()
    return B.lib()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "losa.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(losa_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"losa_select_active", "losa_page_scores_topk", "losa_page_union", "losa_sparse_prefix_attn",
            "losa_block_attn_merge", "losa_update_prefix_cache"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(B.EXPORTS) == set(names)


def shape(**kw):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=1, head_dim=64, block_size=16, page_size=16,
                max_pages_per_seq=64, dtype=0, sm_scale=0.125)
    base.update(kw)
    return B.ShapeT(*[base[k] for k in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "block_size",
                                        "page_size", "max_pages_per_seq", "dtype")], base["sm_scale"])


@pytest.mark.parametrize("kw,code", [
    (dict(), B.LOSA_OK),
    (dict(batch=0), B.LOSA_ERR_INVALID_ARG),
    (dict(block_size=65), B.LOSA_ERR_INVALID_ARG),
    (dict(dtype=7), B.LOSA_ERR_INVALID_ARG),
    (dict(sm_scale=0.0), B.LOSA_ERR_INVALID_ARG),
    (dict(head_dim=96), B.LOSA_ERR_UNSUPPORTED),
    (dict(page_size=48), B.LOSA_ERR_UNSUPPORTED),
    (dict(n_q_heads=5, n_kv_heads=2), B.LOSA_ERR_UNSUPPORTED),
    (dict(n_q_heads=34, n_kv_heads=2), B.LOSA_ERR_UNSUPPORTED),
])
def test_workspace_bytes_validates_shape(lib, kw, code):
    n = C.c_size_t(0)
    s = shape(**kw)
    assert lib.losa_workspace_bytes(C.byref(s), C.byref(n)) == code
    if code == B.LOSA_OK:
        assert n.value > 0 and n.value % 256 == 0


def test_workspace_grows_with_problem(lib):
    a, b = C.c_size_t(0), C.c_size_t(0)
    s1, s2 = shape(), shape(batch=4, max_pages_per_seq=1024, n_q_heads=32, n_kv_heads=8, head_dim=128)
    assert lib.losa_workspace_bytes(C.byref(s1), C.byref(a)) == 0
    assert lib.losa_workspace_bytes(C.byref(s2), C.byref(b)) == 0
    assert b.value > a.value


def test_null_arguments_are_rejected_without_a_device(lib):
    n = C.c_size_t(0)
    assert lib.losa_workspace_bytes(None, C.byref(n)) == B.LOSA_ERR_INVALID_ARG
    assert lib.losa_workspace_bytes(C.byref(shape()), None) == B.LOSA_ERR_INVALID_ARG
    h = C.c_void_p(0)
    assert lib.losa_create(C.byref(shape()), None, C.c_size_t(1 << 20), C.byref(h)) == B.LOSA_ERR_INVALID_ARG
    assert lib.losa_create(C.byref(shape()), C.c_void_p(4096 + 8), C.c_size_t(1 << 20), C.byref(h)) == B.LOSA_ERR_UNSUPPORTED
    assert h.value is None
    assert lib.losa_destroy(None) == B.LOSA_ERR_INVALID_ARG
    assert lib.losa_poll_status(None, None) == B.LOSA_ERR_INVALID_ARG
    for fn, nargs in (("losa_select_active", 10), ("losa_page_scores_topk", 10), ("losa_page_union", 10),
                      ("losa_sparse_prefix_attn", 9), ("losa_block_attn_merge", 8),
                      ("losa_update_prefix_cache", 8), ("losa_build_page_summaries", 3),
                      ("losa_denoise_step_host", 11), ("losa_denoise_step", 12),
                      ("losa_page_scores_topk_pooled", 10), ("losa_page_scores_topk_mma", 10),
                      ("losa_quantize_kv_pages", 4)):
        args = [None] * nargs
        if fn in ("losa_select_active",):
            args[3] = C.c_int32(64)
        assert getattr(lib, fn)(*args) == B.LOSA_ERR_INVALID_ARG, fn
    assert lib.losa_set_pooled_selection(None, C.c_int32(1)) == B.LOSA_ERR_INVALID_ARG
    assert lib.losa_set_wait_limit(None, C.c_int64(5)) == B.LOSA_ERR_INVALID_ARG
    assert lib.losa_set_step_selector(None, C.c_int32(2)) == B.LOSA_ERR_INVALID_ARG
    args = [None] * 11
    args[3], args[4] = C.c_int32(64), C.c_double(0.5)
    assert lib.losa_select_active_tau(*args) == B.LOSA_ERR_INVALID_ARG


def test_missing_library_is_a_loud_error(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/liblosa.so")
    with pytest.raises(ImportError):
        B.lib()
