"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, see losa_oracle.h).

Marshals numpy arrays to `liblosa_oracle.so`; holds no arithmetic of its own.  Element tensors are
`float32` arrays (dtype 0) or `uint16` arrays of bf16 bit patterns (dtype 1).  Only tests, the
smoke check and the benchmark's CPU-baseline leg may import this module; it imports nothing from
the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liblosa_oracle.so")
_SRC = os.path.join(_HERE, "losa_oracle.c")


def build(force: bool = False) -> str:
    """Compiles the oracle with gcc (plain C, OpenMP, no FP contraction, no fast-math)."""
    hdr = os.path.join(_HERE, "losa_oracle.h")
    stale = (not os.path.exists(_SO)) or any(
        os.path.getmtime(f) > os.path.getmtime(_SO) for f in (_SRC, hdr))
    if force or stale:
        subprocess.check_call([
            "gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-Wall", "-shared", "-fPIC",
            "-o", _SO, _SRC, "-lm"])
    return _SO


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "block_size", "page_size",
        "max_pages_per_seq", "dtype")] + [("sm_scale", C.c_double)]


class _KV(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("stride_page", C.c_int64),
                ("stride_head", C.c_int64), ("stride_tok", C.c_int64), ("kmin", C.c_void_p),
                ("kmax", C.c_void_p), ("page_table", C.c_void_p), ("kv_len", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _chk(a, dt, name):
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], name
    assert a.dtype == dt, (name, a.dtype, dt)
    return a


@dataclass
class Shape:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block_size: int
    page_size: int
    max_pages_per_seq: int
    dtype: int  # 0 fp32, 1 bf16 bit patterns
    sm_scale: float

    def c(self):
        return _Shape(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.block_size,
                      self.page_size, self.max_pages_per_seq, self.dtype, self.sm_scale)

    @property
    def elem(self):
        return np.uint16 if self.dtype == 1 else np.float32


class KV:
    """Paged prefix cache on the host: arrays k_pages, v_pages [n_phys, H_kv, g, d], kmin, kmax
    [n_phys, H_kv, d], page_table [N, P_max] int32, kv_len [N] int32."""

    def __init__(self, sh: Shape, k_pages, v_pages, kmin, kmax, page_table, kv_len):
        e = sh.elem
        self.k_pages = _chk(k_pages, e, "k_pages")
        self.v_pages = _chk(v_pages, e, "v_pages")
        self.kmin = _chk(kmin, e, "kmin")
        self.kmax = _chk(kmax, e, "kmax")
        self.page_table = _chk(page_table, np.int32, "page_table")
        self.kv_len = _chk(kv_len, np.int32, "kv_len")
        assert k_pages.shape[1:] == (sh.n_kv_heads, sh.page_size, sh.head_dim)
        assert page_table.shape == (sh.batch, sh.max_pages_per_seq)

    def c(self):
        g, d, hkv = self.k_pages.shape[2], self.k_pages.shape[3], self.k_pages.shape[1]
        return _KV(self.k_pages.ctypes.data, self.v_pages.ctypes.data, hkv * g * d, g * d, d,
                   self.kmin.ctypes.data, self.kmax.ctypes.data, self.page_table.ctypes.data,
                   self.kv_len.ctypes.data)


def build_page_summaries(sh: Shape, kv: KV):
    s, k = sh.c(), kv.c()
    lib().oracle_build_page_summaries(C.byref(s), C.byref(k))


def select_active(sh: Shape, x_cur, x_prev, m_per_seq=None, step=None):
    """Returns (active_idx [N,B] int32, n_active [N] int32, delta [N,B] float64)."""
    N, B = sh.batch, sh.block_size
    x_cur = _chk(x_cur, sh.elem, "x_cur")
    x_prev = _chk(x_prev, sh.elem, "x_prev")
    w = x_cur.size // (N * B)
    act = np.full((N, B), -7, np.int32)
    na = np.zeros(N, np.int32)
    delta = np.zeros((N, B), np.float64)
    m = None if m_per_seq is None else _chk(np.ascontiguousarray(m_per_seq, np.int32), np.int32, "m")
    st = None if step is None else _chk(np.ascontiguousarray(step, np.int32), np.int32, "step")
    s = sh.c()
    lib().oracle_select_active(C.byref(s), _p(x_cur), _p(x_prev), C.c_int32(w), _p(m), _p(st),
                               _p(act), _p(na), _p(delta))
    return act, na, delta


def select_active_tau(sh: Shape, x_cur, x_prev, tau: float, m_cap=None, step=None):
    """Threshold variant of the pruning rule.  Returns (active_idx, n_active, delta) as select_active."""
    N, B = sh.batch, sh.block_size
    x_cur = _chk(x_cur, sh.elem, "x_cur")
    x_prev = _chk(x_prev, sh.elem, "x_prev")
    w = x_cur.size // (N * B)
    act = np.full((N, B), -7, np.int32)
    na = np.zeros(N, np.int32)
    delta = np.zeros((N, B), np.float64)
    m = None if m_cap is None else _chk(np.ascontiguousarray(m_cap, np.int32), np.int32, "m_cap")
    st = None if step is None else _chk(np.ascontiguousarray(step, np.int32), np.int32, "step")
    s = sh.c()
    lib().oracle_select_active_tau(C.byref(s), _p(x_cur), _p(x_prev), C.c_int32(w), C.c_double(tau), _p(m), _p(st),
                                   _p(act), _p(na), _p(delta))
    return act, na, delta


def page_scores_one(sh: Shape, q, kv: KV, s_idx: int, tok: int, head: int):
    """Returns (u32 [P_s] float32 in the fixed order, u64 [P_s] float64)."""
    P = (int(kv.kv_len[s_idx]) + sh.page_size - 1) // sh.page_size
    u32 = np.zeros(P, np.float32)
    u64 = np.zeros(P, np.float64)
    s, k = sh.c(), kv.c()
    lib().oracle_page_scores_one(C.byref(s), _p(_chk(q, sh.elem, "q")), C.byref(k), C.c_int32(s_idx),
                                 C.c_int32(tok), C.c_int32(head), _p(u32), _p(u64))
    return u32, u64


def page_scores_topk(sh: Shape, q, kv: KV, active_idx, n_active, k: int, step=None,
                     topk_pages=None, topk_scores=None):
    """Returns (topk_pages [N,B,H_q,k] int32, topk_scores float32); rows not written keep the
    value they had (a fresh array is filled with -9 / NaN)."""
    N, B, H = sh.batch, sh.block_size, sh.n_q_heads
    if topk_pages is None:
        topk_pages = np.full((N, B, H, k), -9, np.int32)
    if topk_scores is None:
        topk_scores = np.full((N, B, H, k), np.nan, np.float32)
    st = None if step is None else np.ascontiguousarray(step, np.int32)
    s, kk = sh.c(), kv.c()
    lib().oracle_page_scores_topk(C.byref(s), _p(_chk(q, sh.elem, "q")), C.byref(kk),
                                  _p(_chk(active_idx, np.int32, "active_idx")),
                                  _p(_chk(n_active, np.int32, "n_active")), _p(st), C.c_int32(k),
                                  _p(topk_pages), _p(topk_scores))
    return topk_pages, topk_scores


def page_scores_topk_pooled(sh: Shape, q, kv: KV, active_idx, n_active, k: int, step=None,
                            topk_pages=None, topk_scores=None):
    """Selector variant: one list per (token, KV head) from the largest of the G heads' bounds,
    stored for every head of the group.  Same outputs as page_scores_topk."""
    N, B, H = sh.batch, sh.block_size, sh.n_q_heads
    if topk_pages is None:
        topk_pages = np.full((N, B, H, k), -9, np.int32)
    if topk_scores is None:
        topk_scores = np.full((N, B, H, k), np.nan, np.float32)
    st = None if step is None else np.ascontiguousarray(step, np.int32)
    s, kk = sh.c(), kv.c()
    lib().oracle_page_scores_topk_pooled(C.byref(s), _p(_chk(q, sh.elem, "q")), C.byref(kk),
                                         _p(_chk(active_idx, np.int32, "active_idx")),
                                         _p(_chk(n_active, np.int32, "n_active")), _p(st), C.c_int32(k),
                                         _p(topk_pages), _p(topk_scores))
    return topk_pages, topk_scores


def check_topk_relaxed(sh: Shape, q, kv: KV, active_idx, n_active, k: int, topk_pages, eps: float, step=None) -> int:
    """Number of (active token, head) lists that break the relaxed validity rule (fp64 bounds, slack
    eps times the largest sum of term magnitudes); see losa_oracle.c."""
    st = None if step is None else np.ascontiguousarray(step, np.int32)
    s, kvc = sh.c(), kv.c()
    fn = lib().oracle_check_topk_relaxed
    fn.restype = C.c_int64
    return int(fn(C.byref(s), _p(_chk(q, sh.elem, "q")), C.byref(kvc), _p(_chk(active_idx, np.int32, "active_idx")),
                  _p(_chk(n_active, np.int32, "n_active")), _p(st), C.c_int32(k),
                  _p(_chk(topk_pages, np.int32, "topk")), C.c_double(eps)))


# ---- FP8 (E4M3) K/V pages, one power-of-two scale per (physical page, KV head) and tensor
def fp8_decode(codes) -> np.ndarray:
    fn = lib().oracle_fp8_decode
    fn.restype, fn.argtypes = C.c_double, [C.c_uint8]
    return np.array([fn(int(c)) for c in np.asarray(codes, np.uint8).ravel()], np.float64).reshape(np.shape(codes))


def fp8_encode(values) -> np.ndarray:
    fn = lib().oracle_fp8_encode
    fn.restype, fn.argtypes = C.c_uint8, [C.c_double]
    return np.array([fn(float(v)) for v in np.asarray(values, np.float64).ravel()], np.uint8).reshape(np.shape(values))


def fp8_quantize_pages(sh: Shape, kv: KV):
    """Returns (k_codes, v_codes [n_phys,H_kv,g,d] uint8, k_scale, v_scale [n_phys,H_kv] float32) of every logical page."""
    n_phys = kv.k_pages.shape[0]
    shape = (n_phys, sh.n_kv_heads, sh.page_size, sh.head_dim)
    kc, vc = np.zeros(shape, np.uint8), np.zeros(shape, np.uint8)
    ks, vs = np.ones((n_phys, sh.n_kv_heads), np.float32), np.ones((n_phys, sh.n_kv_heads), np.float32)
    s, k = sh.c(), kv.c()
    lib().oracle_fp8_quantize_pages(C.byref(s), C.byref(k), _p(kc), _p(vc), _p(ks), _p(vs))
    return kc, vc, ks, vs


def fp8_dequantize_pages(sh: Shape, k_codes, v_codes, k_scale, v_scale, kv_dst: KV):
    """scale * value(code) of the valid tokens of every logical page into kv_dst's pools (exact in bf16 / fp32)."""
    s, k = sh.c(), kv_dst.c()
    lib().oracle_fp8_dequantize_pages(C.byref(s), _p(_chk(k_codes, np.uint8, "k_codes")), _p(_chk(v_codes, np.uint8, "v_codes")),
                                      _p(_chk(k_scale, np.float32, "k_scale")), _p(_chk(v_scale, np.float32, "v_scale")), C.byref(k))


def fp8_append_block(sh: Shape, page_table, kv_len, k_codes, v_codes, k_scale, v_scale, k_blk, v_blk):
    """Appends the block to the FP8 cache (re-quantising every touched page) and adds B to kv_len, in place."""
    s = sh.c()
    lib().oracle_fp8_append_block(C.byref(s), _p(_chk(page_table, np.int32, "page_table")), _p(_chk(kv_len, np.int32, "kv_len")),
                                  _p(_chk(k_codes, np.uint8, "k_codes")), _p(_chk(v_codes, np.uint8, "v_codes")),
                                  _p(_chk(k_scale, np.float32, "k_scale")), _p(_chk(v_scale, np.float32, "v_scale")),
                                  _p(_chk(k_blk, sh.elem, "k_blk")), _p(_chk(v_blk, sh.elem, "v_blk")))


def round_bf16(x) -> np.ndarray:
    """Element-wise rounding to bf16 (ties to even) of float64 values, as float64."""
    lib().oracle_round_bf16.restype = C.c_double
    lib().oracle_round_bf16.argtypes = [C.c_double]
    v = np.asarray(x, np.float64)
    return np.array([lib().oracle_round_bf16(float(t)) for t in v.ravel()], np.float64).reshape(v.shape)


def round_state_bf16(sh: Shape, o_p, active_idx, n_active):
    """bf16 state: rounds the rows of the active tokens of o_p (float64 [N, B, H_q, d]) in place."""
    s = sh.c()
    lib().oracle_round_state_bf16(C.byref(s), _p(_chk(o_p, np.float64, "o_p")), _p(_chk(active_idx, np.int32, "active_idx")),
                                  _p(_chk(n_active, np.int32, "n_active")))


def page_union(sh: Shape, topk_pages, active_idx, n_active, k: int, kv_len, step=None):
    """Returns (union_pages [N,H_kv,P_max] int32, union_count [N,H_kv] int32)."""
    N, Hkv, P = sh.batch, sh.n_kv_heads, sh.max_pages_per_seq
    up = np.full((N, Hkv, P), -9, np.int32)
    uc = np.zeros((N, Hkv), np.int32)
    st = None if step is None else np.ascontiguousarray(step, np.int32)
    s = sh.c()
    lib().oracle_page_union(C.byref(s), _p(_chk(topk_pages, np.int32, "topk")),
                            _p(_chk(active_idx, np.int32, "active_idx")),
                            _p(_chk(n_active, np.int32, "n_active")), C.c_int32(k),
                            _p(_chk(kv_len, np.int32, "kv_len")), _p(st), _p(up), _p(uc))
    return up, uc


def sparse_prefix_attn(sh: Shape, q, kv: KV, active_idx, n_active, union_pages, union_count,
                       o_p, lse_p):
    """Updates o_p [N,B,H_q,d] float64 and lse_p [N,B,H_q] float64 in place for active tokens."""
    s, k = sh.c(), kv.c()
    _chk(o_p, np.float64, "o_p")
    _chk(lse_p, np.float64, "lse_p")
    lib().oracle_sparse_prefix_attn(C.byref(s), _p(_chk(q, sh.elem, "q")), C.byref(k),
                                    _p(_chk(active_idx, np.int32, "active_idx")),
                                    _p(_chk(n_active, np.int32, "n_active")),
                                    _p(_chk(union_pages, np.int32, "union_pages")),
                                    _p(_chk(union_count, np.int32, "union_count")), _p(o_p),
                                    _p(lse_p))


def block_attn_merge(sh: Shape, q, k_blk, v_blk, o_p, lse_p):
    """Returns (out [N,B,H_q,d] float64, lse [N,B,H_q] float64)."""
    N, B, H, d = sh.batch, sh.block_size, sh.n_q_heads, sh.head_dim
    out = np.zeros((N, B, H, d), np.float64)
    lse = np.zeros((N, B, H), np.float64)
    s = sh.c()
    lib().oracle_block_attn_merge(C.byref(s), _p(_chk(q, sh.elem, "q")),
                                  _p(_chk(k_blk, sh.elem, "k_blk")), _p(_chk(v_blk, sh.elem, "v_blk")),
                                  _p(_chk(o_p, np.float64, "o_p")), _p(_chk(lse_p, np.float64, "lse_p")),
                                  _p(out), _p(lse))
    return out, lse


def update_prefix_cache(sh: Shape, kv: KV, q_prev, step, q, k_blk, v_blk, finalize_block: bool):
    s, k = sh.c(), kv.c()
    lib().oracle_update_prefix_cache(C.byref(s), C.byref(k), _p(_chk(q_prev, sh.elem, "q_prev")),
                                     _p(_chk(step, np.int32, "step")), _p(_chk(q, sh.elem, "q")),
                                     _p(_chk(k_blk, sh.elem, "k_blk")),
                                     _p(_chk(v_blk, sh.elem, "v_blk")),
                                     C.c_int32(1 if finalize_block else 0))
