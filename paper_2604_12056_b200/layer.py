"""Device buffers of one attention layer and the per-step call sequence of include/losa.h.

Convenience for tests and benchmarks: allocation (torch) and the order of the six C-ABI calls.
No arithmetic happens here; every stage runs in the CUDA library.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def to_device(a: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy float32 / int32 / uint16-as-bf16 array -> CUDA tensor (bf16 for uint16 input)."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host(t: torch.Tensor) -> np.ndarray:
    """CUDA tensor -> numpy (bf16 comes back as float32 values)."""
    t = t.detach().cpu()
    return t.float().numpy() if t.dtype == torch.bfloat16 else t.numpy()


class LosaLayer:
    """One layer's paged KV pool, LoSA cache and scratch index buffers on the GPU.

    mode "losa" runs the method; "naive" keeps every token active (per-query sparse attention over
    the whole block); "dense" pins the step counter seen by stages 1-3 to zero (dense prefix
    attention every step).
    """

    def __init__(self, cfg, k_pages, v_pages, page_table, kv_len, mode="losa", device="cuda",
                 share_pool_with: "LosaLayer | None" = None, tau: float = 0.0, pooled: bool = False,
                 mma_selector: bool = False, fp8_kv: bool = False, state_bf16: bool = False):
        self.cfg, self.mode, self.device = cfg, mode, device
        self.tau = tau            # > 0: stage 1 keeps tokens until their Delta reach tau of the block's total
        self.pooled = pooled      # stage 2 keeps one page list per (token, KV head) instead of one per query head
        self.mma_selector = mma_selector   # stage 2 takes its scores from the tensor cores (relaxed list rule, bf16)
        N, Bk, Hq, Hkv, d = cfg.batch, cfg.block_size, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        self.dtype = B.LOSA_BF16 if cfg.dtype == "bf16" else B.LOSA_F32
        td = B.torch_dtype(self.dtype)
        Pmax = cfg.max_pages_per_seq
        self.ctx = B.Context(N, Hq, Hkv, d, Bk, cfg.page_size, Pmax, self.dtype, cfg.sm_scale, device)
        if pooled:
            self.ctx.set_pooled_selection(True)
        if mma_selector and self.dtype == B.LOSA_BF16:
            self.ctx.set_step_selector(2)              # the whole-step call takes the tensor-core selector as well
        if share_pool_with is not None:
            o = share_pool_with
            self.k_pages, self.v_pages, self.kmin, self.kmax = o.k_pages, o.v_pages, o.kmin, o.kmax
            self.page_table = o.page_table
        else:
            self.k_pages = k_pages if isinstance(k_pages, torch.Tensor) else to_device(k_pages, device)
            self.v_pages = v_pages if isinstance(v_pages, torch.Tensor) else to_device(v_pages, device)
            n_phys = self.k_pages.shape[0]
            self.kmin = torch.zeros((n_phys, Hkv, d), dtype=td, device=device)
            self.kmax = torch.zeros((n_phys, Hkv, d), dtype=td, device=device)
            self.page_table = page_table if isinstance(page_table, torch.Tensor) else to_device(page_table, device)
        self.kv_len = (kv_len.clone() if isinstance(kv_len, torch.Tensor) else to_device(kv_len, device))
        self.kv = B.make_kv(self.k_pages, self.v_pages, self.kmin, self.kmax, self.page_table, self.kv_len)
        self.fp8_kv = fp8_kv
        if fp8_kv:
            # FP8 (E4M3) cache with one power-of-two scale per (page, KV head): quantised from the bf16
            # pools by the library, which also writes the summaries of the dequantised keys; every
            # stage then works on the FP8 cache (the bf16 pools can be released by the caller)
            assert share_pool_with is None and self.dtype == B.LOSA_BF16
            n_phys = self.k_pages.shape[0]
            self.k_codes = torch.zeros(self.k_pages.shape, dtype=torch.uint8, device=device)
            self.v_codes = torch.zeros(self.v_pages.shape, dtype=torch.uint8, device=device)
            self.k_scale = torch.ones((n_phys, Hkv), dtype=torch.float32, device=device)
            self.v_scale = torch.ones((n_phys, Hkv), dtype=torch.float32, device=device)
            self.kv_native = self.kv
            self.kv = B.make_kv(self.k_codes, self.v_codes, self.kmin, self.kmax, self.page_table, self.kv_len,
                                self.k_scale, self.v_scale)
        self.q_prev = torch.zeros((N, Bk, Hq, d), dtype=td, device=device)
        # cached prefix output: fp32, or stored rounded to bf16 (bf16 contexts only)
        self.o_p = torch.zeros((N, Bk, Hq, d), dtype=torch.bfloat16 if state_bf16 else torch.float32, device=device)
        self.lse_p = torch.zeros((N, Bk, Hq), dtype=torch.float32, device=device)
        self.step = torch.zeros(N, dtype=torch.int32, device=device)
        self.zero_step = torch.zeros(N, dtype=torch.int32, device=device)
        self.state = B.make_state(self.q_prev, self.o_p, self.lse_p, self.step)
        k = cfg.topk
        self.active_idx = torch.full((N, Bk), -1, dtype=torch.int32, device=device)
        self.n_active = torch.zeros(N, dtype=torch.int32, device=device)
        self.delta = torch.zeros((N, Bk), dtype=torch.float32, device=device)
        self.topk_pages = torch.full((N, Bk, Hq, k), -9, dtype=torch.int32, device=device)
        self.topk_scores = torch.full((N, Bk, Hq, k), float("nan"), dtype=torch.float32, device=device)
        self.union_pages = torch.full((N, Hkv, max(Pmax, 1)), -9, dtype=torch.int32, device=device)
        self.union_count = torch.zeros((N, Hkv), dtype=torch.int32, device=device)
        self.out = torch.zeros((N, Bk, Hq, d), dtype=td, device=device)
        self.lse_out = torch.zeros((N, Bk, Hq), dtype=torch.float32, device=device)
        if fp8_kv:
            B.losa_quantize_kv_pages(self.ctx, self.kv_native, self.kv)
        elif share_pool_with is None:
            B.losa_build_page_summaries(self.ctx, self.kv)

    def stage_step_arg(self):
        return self.zero_step if self.mode == "dense" else self.step

    def run_step(self, q, k_blk, v_blk, m_per_seq, x_sel=None, want_scores=False):
        """Enqueues stages 1-6 for one layer-step on the current stream.  q, k_blk, v_blk and
        m_per_seq are CUDA tensors; x_sel = (x_cur, x_prev) replaces the queries in stage 1."""
        c, cfg = self.ctx, self.cfg
        st = self.stage_step_arg()
        m = None if self.mode == "naive" else m_per_seq
        xc, xp = (q, self.q_prev) if x_sel is None else x_sel
        row_width = xc.numel() // (cfg.batch * cfg.block_size)
        if self.tau > 0.0 and self.mode == "losa":
            B.losa_select_active_tau(c, xc, xp, row_width, self.tau, None, st, self.active_idx, self.n_active, self.delta)
        else:
            B.losa_select_active(c, xc, xp, row_width, m, st, self.active_idx, self.n_active, self.delta)
        scores_topk = (B.losa_page_scores_topk_mma if self.mma_selector else
                       B.losa_page_scores_topk_pooled if self.pooled else B.losa_page_scores_topk)
        scores_topk(c, q, self.kv, self.active_idx, self.n_active, st, cfg.topk, self.topk_pages,
                    self.topk_scores if want_scores else None)
        B.losa_page_union(c, self.topk_pages, self.active_idx, self.n_active, cfg.topk, self.kv_len, st,
                          self.union_pages, self.union_count)
        B.losa_sparse_prefix_attn(c, q, self.kv, self.active_idx, self.n_active, self.union_pages,
                                  self.union_count, self.state)
        B.losa_block_attn_merge(c, q, k_blk, v_blk, self.state, self.out, self.lse_out)
        B.losa_update_prefix_cache(c, self.kv, self.state, q, k_blk, v_blk, False)

    def run_step_fused(self, q, k_blk, v_blk, m_per_seq):
        """The same layer-step through the single whole-step entry point (losa_denoise_step)."""
        if self.mode != "losa":
            raise ValueError("the whole-step call implements the method itself; baselines use run_step")
        if not hasattr(self, "_step_buf"):
            self._step_buf = B.StepBuffersT(0, 0, 0, 0, self.active_idx.data_ptr(), self.n_active.data_ptr(),
                                            self.topk_pages.data_ptr(), self.union_pages.data_ptr(),
                                            self.union_count.data_ptr())
        B.losa_denoise_step(self.ctx, q, k_blk, v_blk, self.out, self.lse_out, self.kv, self.state,
                            self._step_buf, m_per_seq, self.cfg.topk)

    def finalize_block(self, k_blk, v_blk):
        B.losa_update_prefix_cache(self.ctx, self.kv, self.state, None, k_blk, v_blk, True)

    def snapshot(self):
        """Host copies of every intermediate of the last step."""
        return dict(act=to_host(self.active_idx), na=to_host(self.n_active), delta=to_host(self.delta),
                    topk=to_host(self.topk_pages), topk_scores=to_host(self.topk_scores),
                    up=to_host(self.union_pages), uc=to_host(self.union_count), o_p=to_host(self.o_p.float()),
                    lse_p=to_host(self.lse_p), out=to_host(self.out), lse=to_host(self.lse_out),
                    step=to_host(self.step), kv_len=to_host(self.kv_len))
