"""ctypes binding of the C-ABI library declared in include/losa.h.

Argument marshalling only: every function below has the name and the arguments of the C entry
point, takes `torch` CUDA tensors where the C call takes device pointers, and enqueues on the
current torch stream.  There is no CPU fallback — if `liblosa.so` is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblosa.so")

LOSA_OK = 0
LOSA_ERR_INVALID_ARG = -1
LOSA_ERR_UNSUPPORTED = -2
LOSA_ERR_CUDA = -3
LOSA_ERR_TIMEOUT = -4
LOSA_ERR_BOUNDS = -5
LOSA_F32, LOSA_BF16 = 0, 1

EXPORTS = [
    "losa_workspace_bytes", "losa_create", "losa_destroy", "losa_poll_status",
    "losa_last_cuda_error", "losa_launch_count", "losa_select_active", "losa_page_scores_topk",
    "losa_page_union", "losa_sparse_prefix_attn", "losa_block_attn_merge",
    "losa_update_prefix_cache", "losa_build_page_summaries", "losa_denoise_step_host",
    "losa_profile_stage4", "losa_stage4_last_ms", "losa_select_active_static",
    "losa_denoise_step", "losa_select_active_tau", "losa_page_scores_topk_pooled",
    "losa_set_pooled_selection", "losa_set_step_selector", "losa_set_wait_limit", "losa_page_scores_topk_mma", "losa_quantize_kv_pages",
]


class LosaError(RuntimeError):
    def __init__(self, call, code, cuda=0):
        names = {-1: "INVALID_ARG", -2: "UNSUPPORTED", -3: "CUDA", -4: "TIMEOUT", -5: "BOUNDS"}
        super().__init__(f"{call} failed: LOSA_ERR_{names.get(code, code)}" + (f" (cuda error {cuda})" if cuda else ""))
        self.code = code


class ShapeT(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "block_size", "page_size",
        "max_pages_per_seq", "dtype")] + [("sm_scale", C.c_float)]


class KvT(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("stride_page", C.c_int64),
                ("stride_head", C.c_int64), ("stride_tok", C.c_int64), ("kmin", C.c_void_p),
                ("kmax", C.c_void_p), ("page_table", C.c_void_p), ("kv_len", C.c_void_p),
                ("n_phys_pages", C.c_int32), ("kv_format", C.c_int32), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p)]


class StateT(C.Structure):
    _fields_ = [("q_prev", C.c_void_p), ("o_p", C.c_void_p), ("lse_p", C.c_void_p), ("step", C.c_void_p),
                ("o_p_format", C.c_int32)]


class StepBuffersT(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("d_q", "d_k_blk", "d_v_blk", "d_out", "active_idx", "n_active",
                                          "topk_pages", "union_pages", "union_count")]


_lib = None


def lib() -> C.CDLL:
    """Loads liblosa.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2604_12056_b200.build`")
        _lib = C.CDLL(LIB_PATH)
        for n in EXPORTS:
            getattr(_lib, n).restype = C.c_int32
        _lib.losa_launch_count.restype = C.c_int64
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _hptr(t):
    assert isinstance(t, torch.Tensor) and not t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def torch_dtype(dtype: int):
    return torch.bfloat16 if dtype == LOSA_BF16 else torch.float32


LOSA_KV_NATIVE, LOSA_KV_FP8_E4M3 = 0, 1


def make_kv(k_pages, v_pages, kmin, kmax, page_table, kv_len, k_scale=None, v_scale=None) -> KvT:
    """losa_kv_t over a [n_phys, H_kv, g, d] pool (any strides with contiguous token rows).  With
    k_scale / v_scale ([n_phys, H_kv] fp32) the pools are uint8 tensors of E4M3 codes."""
    sp, sh_, st, sd = k_pages.stride()
    assert sd == 1 and v_pages.stride() == k_pages.stride()
    fp8 = k_scale is not None
    assert (k_pages.dtype == torch.uint8) == fp8
    kv = KvT(k_pages.data_ptr(), v_pages.data_ptr(), sp, sh_, st,
             0 if kmin is None else kmin.data_ptr(), 0 if kmax is None else kmax.data_ptr(),
             page_table.data_ptr(), kv_len.data_ptr(), k_pages.shape[0],
             LOSA_KV_FP8_E4M3 if fp8 else LOSA_KV_NATIVE, k_scale.data_ptr() if fp8 else 0, v_scale.data_ptr() if fp8 else 0)
    kv._keep = (k_pages, v_pages, kmin, kmax, page_table, kv_len, k_scale, v_scale)
    return kv


LOSA_STATE_F32, LOSA_STATE_BF16 = 0, 1


def make_state(q_prev, o_p, lse_p, step) -> StateT:
    """o_p: float32, or bfloat16 for the bf16 state (stored rounded; bf16 contexts only)."""
    import torch
    fmt = LOSA_STATE_BF16 if o_p.dtype == torch.bfloat16 else LOSA_STATE_F32
    st = StateT(q_prev.data_ptr(), o_p.data_ptr(), lse_p.data_ptr(), step.data_ptr(), fmt)
    st._keep = (q_prev, o_p, lse_p, step)
    return st


class Context:
    """losa_ctx plus its caller-owned workspace (a torch tensor)."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, block_size, page_size,
                 max_pages_per_seq, dtype, sm_scale, device="cuda"):
        self.shape = ShapeT(batch, n_q_heads, n_kv_heads, head_dim, block_size, page_size,
                            max_pages_per_seq, dtype, sm_scale)
        with torch.cuda.device(device):
            n = C.c_size_t(0)
            self._check("losa_workspace_bytes", lib().losa_workspace_bytes(C.byref(self.shape), C.byref(n)))
            self.workspace_bytes = int(n.value)
            self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=device)
            off = (-self.workspace.data_ptr()) % 256
            self._ws_ptr = self.workspace.data_ptr() + off
            h = C.c_void_p(0)
            self._h = None
            self._check("losa_create", lib().losa_create(C.byref(self.shape), C.c_void_p(self._ws_ptr),
                                                          C.c_size_t(self.workspace_bytes), C.byref(h)))
            self._h = h

    def _check(self, call, rc):
        if rc != LOSA_OK:
            cuda = lib().losa_last_cuda_error(self._h) if getattr(self, "_h", None) else 0
            raise LosaError(call, rc, cuda)

    def close(self):
        if self._h is not None:
            lib().losa_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def launch_count(self) -> int:
        return int(lib().losa_launch_count(self._h))

    def set_step_selector(self, selector: int):
        """0 = exact per-head lists, 1 = pooled per KV head, 2 = tensor-core scores (relaxed list rule)."""
        self._check("losa_set_step_selector", lib().losa_set_step_selector(self._h, C.c_int32(selector)))

    def set_pooled_selection(self, on: bool):
        self._check("losa_set_pooled_selection", lib().losa_set_pooled_selection(self._h, C.c_int32(1 if on else 0)))

    def set_wait_limit(self, cycles: int):
        """Bound of the bf16 stage-4 kernel's internal waits in SM clock cycles; <= 0 restores the default."""
        self._check("losa_set_wait_limit", lib().losa_set_wait_limit(self._h, C.c_int64(int(cycles))))

    def profile_stage4(self, enable: bool):
        self._check("losa_profile_stage4", lib().losa_profile_stage4(self._h, C.c_int32(1 if enable else 0)))

    def stage4_last_ms(self) -> float:
        ms = C.c_float(0.0)
        self._check("losa_stage4_last_ms", lib().losa_stage4_last_ms(self._h, C.byref(ms)))
        return float(ms.value)

    def poll_status(self) -> int:
        return int(lib().losa_poll_status(self._h, _stream()))


def losa_select_active(ctx, x_cur, x_prev, row_width, m_per_seq, step, active_idx, n_active, delta_opt=None):
    ctx._check("losa_select_active", lib().losa_select_active(
        ctx._h, _ptr(x_cur), _ptr(x_prev), C.c_int32(row_width), _ptr(m_per_seq), _ptr(step),
        _ptr(active_idx), _ptr(n_active), _ptr(delta_opt), _stream()))


def losa_select_active_tau(ctx, x_cur, x_prev, row_width, tau, m_cap_opt, step, active_idx, n_active, delta_opt=None):
    """Stage 1, threshold variant: tokens are kept until their Delta reach tau of the block's total."""
    ctx._check("losa_select_active_tau", lib().losa_select_active_tau(
        ctx._h, _ptr(x_cur), _ptr(x_prev), C.c_int32(row_width), C.c_double(tau), _ptr(m_cap_opt), _ptr(step),
        _ptr(active_idx), _ptr(n_active), _ptr(delta_opt), _stream()))


def losa_select_active_static(shape: ShapeT, x_cur, x_prev, row_width, m_per_seq, step, active_idx, n_active,
                              delta_opt=None):
    """Stage 1 for callers that must not allocate device memory: no context, no workspace; the
    scratch lives in a fixed array inside the library (batch <= 64).  Calls on one device share
    that array, so they must not overlap on the GPU."""
    rc = lib().losa_select_active_static(C.byref(shape), _ptr(x_cur), _ptr(x_prev), C.c_int32(row_width),
                                         _ptr(m_per_seq), _ptr(step), _ptr(active_idx), _ptr(n_active),
                                         _ptr(delta_opt), _stream())
    if rc != LOSA_OK:
        raise LosaError("losa_select_active_static", rc)


def losa_page_scores_topk(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt=None):
    ctx._check("losa_page_scores_topk", lib().losa_page_scores_topk(
        ctx._h, _ptr(q), C.byref(kv), _ptr(active_idx), _ptr(n_active), _ptr(step), C.c_int32(k),
        _ptr(topk_pages), _ptr(topk_scores_opt), _stream()))


def losa_page_scores_topk_pooled(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt=None):
    ctx._check("losa_page_scores_topk_pooled", lib().losa_page_scores_topk_pooled(
        ctx._h, _ptr(q), C.byref(kv), _ptr(active_idx), _ptr(n_active), _ptr(step), C.c_int32(k),
        _ptr(topk_pages), _ptr(topk_scores_opt), _stream()))


def losa_page_scores_topk_mma(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt=None):
    """Stage 2 with tensor-core scores (bf16): lists valid under the relaxed rule, not entry by entry."""
    ctx._check("losa_page_scores_topk_mma", lib().losa_page_scores_topk_mma(
        ctx._h, _ptr(q), C.byref(kv), _ptr(active_idx), _ptr(n_active), _ptr(step), C.c_int32(k),
        _ptr(topk_pages), _ptr(topk_scores_opt), _stream()))


def losa_page_union(ctx, topk_pages, active_idx, n_active, k, kv_len, step, union_pages, union_count):
    ctx._check("losa_page_union", lib().losa_page_union(
        ctx._h, _ptr(topk_pages), _ptr(active_idx), _ptr(n_active), C.c_int32(k), _ptr(kv_len), _ptr(step),
        _ptr(union_pages), _ptr(union_count), _stream()))


def losa_sparse_prefix_attn(ctx, q, kv, active_idx, n_active, union_pages, union_count, state):
    ctx._check("losa_sparse_prefix_attn", lib().losa_sparse_prefix_attn(
        ctx._h, _ptr(q), C.byref(kv), _ptr(active_idx), _ptr(n_active), _ptr(union_pages),
        _ptr(union_count), C.byref(state), _stream()))


def losa_block_attn_merge(ctx, q, k_blk, v_blk, state, out, lse_out_opt=None):
    ctx._check("losa_block_attn_merge", lib().losa_block_attn_merge(
        ctx._h, _ptr(q), _ptr(k_blk), _ptr(v_blk), C.byref(state), _ptr(out), _ptr(lse_out_opt), _stream()))


def losa_update_prefix_cache(ctx, kv, state, q, k_blk, v_blk, finalize_block):
    ctx._check("losa_update_prefix_cache", lib().losa_update_prefix_cache(
        ctx._h, C.byref(kv), C.byref(state), _ptr(q), _ptr(k_blk), _ptr(v_blk),
        C.c_int32(1 if finalize_block else 0), _stream()))


def losa_quantize_kv_pages(ctx, src_kv, dst_kv):
    """bf16 cache -> FP8 cache (codes, per-page scales, summaries of the dequantised keys)."""
    ctx._check("losa_quantize_kv_pages", lib().losa_quantize_kv_pages(ctx._h, C.byref(src_kv), C.byref(dst_kv), _stream()))


def losa_build_page_summaries(ctx, kv):
    ctx._check("losa_build_page_summaries", lib().losa_build_page_summaries(ctx._h, C.byref(kv), _stream()))


def losa_denoise_step(ctx, q, k_blk, v_blk, out, lse_out_opt, kv, state, buf, m_per_seq, k):
    ctx._check("losa_denoise_step", lib().losa_denoise_step(
        ctx._h, _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out), _ptr(lse_out_opt), C.byref(kv), C.byref(state),
        C.byref(buf), _ptr(m_per_seq), C.c_int32(k), _stream()))


def losa_denoise_step_host(ctx, h_q, h_k_blk, h_v_blk, h_out, kv, state, buf, m_per_seq, k):
    ctx._check("losa_denoise_step_host", lib().losa_denoise_step_host(
        ctx._h, _hptr(h_q), _hptr(h_k_blk), _hptr(h_v_blk), _hptr(h_out), C.byref(kv), C.byref(state),
        C.byref(buf), _ptr(m_per_seq), C.c_int32(k), _stream()))
