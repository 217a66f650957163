"""Shared test utilities: tiny random problems laid out like the library's interface, and
brute-force reference routines written directly from the definitions (numpy fp64 / torch fp64).

Nothing here is used by the product path.
"""
from __future__ import annotations

import numpy as np

from oracle import oracle as orc
from paper_2604_12056_b200 import workloads as wl


def make_shape(N, Hq, Hkv, d, B, g, Pmax, dtype="f32", sm_scale=None):
    return orc.Shape(N, Hq, Hkv, d, B, g, Pmax, 1 if dtype == "bf16" else 0,
                     float(1.0 / np.sqrt(d)) if sm_scale is None else float(sm_scale))


class Problem:
    """A small paged problem with plain (logical-order) copies kept for brute-force checks."""

    def __init__(self, seed, N=1, Hq=4, Hkv=2, d=16, B=4, g=4, kv_lens=(10,), dtype="f32",
                 extra_pages=2, scale=1.0, pad_nan=True, shuffle=True):
        rng = np.random.default_rng(seed)
        self.rng = rng
        self.dtype = dtype
        kv_lens = tuple(kv_lens)
        assert len(kv_lens) == N
        Pmax = max((L + g - 1) // g for L in kv_lens) + extra_pages
        self.sh = make_shape(N, Hq, Hkv, d, B, g, Pmax, dtype)
        n_phys = N * Pmax
        perm = rng.permutation(n_phys) if shuffle else np.arange(n_phys)
        self.page_table = np.ascontiguousarray(perm.reshape(N, Pmax).astype(np.int32))
        self.kv_len = np.asarray(kv_lens, np.int32)
        # logical fp32 copies [N][L, Hkv, d]
        self.K = [self._round(scale * rng.standard_normal((L, Hkv, d)).astype(np.float32)) for L in kv_lens]
        self.V = [self._round(rng.standard_normal((L, Hkv, d)).astype(np.float32)) for L in kv_lens]
        fill = np.nan if pad_nan else 0.0
        kp = np.full((n_phys, Hkv, g, d), fill, np.float32)
        vp = np.full((n_phys, Hkv, g, d), fill, np.float32)
        for s, L in enumerate(kv_lens):
            for t in range(L):
                ph = self.page_table[s, t // g]
                kp[ph, :, t % g, :] = self.K[s][t]
                vp[ph, :, t % g, :] = self.V[s][t]
        self.k_pages = wl.to_elem(kp, dtype)
        self.v_pages = wl.to_elem(vp, dtype)
        e = self.k_pages.dtype
        self.kmin = np.zeros((n_phys, Hkv, d), e)
        self.kmax = np.zeros((n_phys, Hkv, d), e)
        self.kv = orc.KV(self.sh, self.k_pages, self.v_pages, self.kmin, self.kmax,
                         self.page_table, self.kv_len)
        self.q = self.rand_elem((N, B, Hq, d), scale)
        self.k_blk = self.rand_elem((N, B, Hkv, d), scale)
        self.v_blk = self.rand_elem((N, B, Hkv, d))

    def _round(self, x):
        return wl.elem_to_f32(wl.to_elem(x, self.dtype))

    def rand_elem(self, shape, scale=1.0):
        return wl.to_elem(scale * self.rng.standard_normal(shape).astype(np.float32), self.dtype)

    def f(self, x):
        """Element array -> float64 values."""
        return wl.elem_to_f32(x).astype(np.float64)

    def pages(self, s):
        return (int(self.kv_len[s]) + self.sh.page_size - 1) // self.sh.page_size


def softmax_attention(q, K, V, scale):
    """Textbook attention of one query row over rows of K, V (fp64): softmax(scale q K^T) V, and
    the log-sum-exp of the scaled scores.  Two passes, no online tricks."""
    q, K, V = np.asarray(q, np.float64), np.asarray(K, np.float64), np.asarray(V, np.float64)
    if K.shape[0] == 0:
        return np.zeros(V.shape[1]), -np.inf
    s = scale * (K @ q)
    m = s.max()
    w = np.exp(s - m)
    return (w / w.sum()) @ V, m + np.log(w.sum())


def torch_sdpa(q, K, V, scale):
    """Same through torch's scaled_dot_product_attention in fp64 (a library routine)."""
    import torch
    import torch.nn.functional as F
    qq = torch.from_numpy(np.asarray(q, np.float64))[None, None, None, :]
    kk = torch.from_numpy(np.asarray(K, np.float64))[None, None]
    vv = torch.from_numpy(np.asarray(V, np.float64))[None, None]
    return F.scaled_dot_product_attention(qq, kk, vv, scale=scale)[0, 0, 0].numpy()


# ---------------------------------------------------------------- whole denoising blocks, oracle side
def oracle_shape_of(cfg):
    return orc.Shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.block_size,
                     cfg.page_size, cfg.max_pages_per_seq, 1 if cfg.dtype == "bf16" else 0,
                     cfg.sm_scale)


class OracleLayer:
    """Host-side state of one attention layer driven through the oracle, step by step.

    mode "losa": the paper's method; "naive": every token active every step (per-query sparse
    attention applied to the whole block, Section 5.1 baselines); "dense": step counter pinned to
    0, i.e. dense prefix attention every step."""

    def __init__(self, w, mode="losa", tau=0.0, pooled=False, state_bf16=False):
        self.tau = tau
        self.pooled = pooled
        self.state_bf16 = state_bf16      # the cached prefix output is stored rounded to bf16
        cfg = w.cfg
        self.w, self.cfg, self.mode = w, cfg, mode
        self.sh = oracle_shape_of(cfg)
        e = w.k_pages.dtype
        self.k_pages, self.v_pages = w.k_pages.copy(), w.v_pages.copy()
        self.kv_len = w.kv_len.copy()
        self.kmin = np.zeros((w.n_phys, cfg.n_kv_heads, cfg.head_dim), e)
        self.kmax = np.zeros_like(self.kmin)
        self.kv = orc.KV(self.sh, self.k_pages, self.v_pages, self.kmin, self.kmax,
                         w.page_table, self.kv_len)
        orc.build_page_summaries(self.sh, self.kv)
        N, B, H, d = cfg.batch, cfg.block_size, cfg.n_q_heads, cfg.head_dim
        self.q_prev = np.zeros((N, B, H, d), e)
        self.o_p = np.zeros((N, B, H, d), np.float64)
        self.lse_p = np.zeros((N, B, H), np.float64)
        self.step = np.zeros(N, np.int32)
        self.topk = np.full((N, B, H, cfg.topk), -9, np.int32)

    def run_step(self, inp, x_sel=None, finalize=False):
        """One layer-step; returns every intermediate.  x_sel: (cur, prev) to drive Eq. 1 with
        something other than the queries."""
        sh, cfg = self.sh, self.cfg
        step = np.zeros_like(self.step) if self.mode == "dense" else self.step
        m = None if self.mode == "naive" else inp.m_per_seq
        xc, xp = (inp.q, self.q_prev) if x_sel is None else x_sel
        if self.tau > 0.0 and self.mode == "losa":
            act, na, delta = orc.select_active_tau(sh, xc, xp, self.tau, None, step)
        else:
            act, na, delta = orc.select_active(sh, xc, xp, m, step)
        scores_topk = orc.page_scores_topk_pooled if self.pooled else orc.page_scores_topk
        scores_topk(sh, inp.q, self.kv, act, na, cfg.topk, step, topk_pages=self.topk)
        up, uc = orc.page_union(sh, self.topk, act, na, cfg.topk, self.kv_len, step)
        orc.sparse_prefix_attn(sh, inp.q, self.kv, act, na, up, uc, self.o_p, self.lse_p)
        if self.state_bf16:
            orc.round_state_bf16(sh, self.o_p, act, na)
        out, lse = orc.block_attn_merge(sh, inp.q, inp.k_blk, inp.v_blk, self.o_p, self.lse_p)
        res = dict(act=act, na=na, delta=delta, topk=self.topk.copy(), up=up, uc=uc,
                   o_p=self.o_p.copy(), lse_p=self.lse_p.copy(), out=out, lse=lse,
                   step_before=self.step.copy())
        orc.update_prefix_cache(sh, self.kv, self.q_prev, self.step, inp.q, inp.k_blk, inp.v_blk, False)
        if finalize:
            orc.update_prefix_cache(sh, self.kv, self.q_prev, self.step, inp.q, inp.k_blk, inp.v_blk, True)
        return res


class OracleFp8Layer(OracleLayer):
    """The same layer over an FP8 (E4M3) cache: the oracle quantises the workload's pools page by page
    (its own quantiser), and every stage then runs - unchanged - on the dequantised values, which are
    exact in the element type.  Block finalisation appends through the FP8 rule (touched pages are
    re-quantised) and refreshes the dequantised copy and the summaries."""

    def __init__(self, w, mode="losa", **kw):
        import types
        cfg = w.cfg
        sh = oracle_shape_of(cfg)
        e = w.k_pages.dtype
        kmin = np.zeros((w.n_phys, cfg.n_kv_heads, cfg.head_dim), e)
        kv_src = orc.KV(sh, w.k_pages, w.v_pages, kmin, kmin.copy(), w.page_table, w.kv_len.copy())
        self.k_codes, self.v_codes, self.k_scale, self.v_scale = orc.fp8_quantize_pages(sh, kv_src)
        deq = types.SimpleNamespace(cfg=cfg, k_pages=np.zeros_like(w.k_pages), v_pages=np.zeros_like(w.v_pages),
                                    page_table=w.page_table, kv_len=w.kv_len.copy(), n_phys=w.n_phys)
        kv_dst = orc.KV(sh, deq.k_pages, deq.v_pages, kmin.copy(), kmin.copy(), w.page_table, deq.kv_len)
        orc.fp8_dequantize_pages(sh, self.k_codes, self.v_codes, self.k_scale, self.v_scale, kv_dst)
        super().__init__(deq, mode, **kw)

    def run_step(self, inp, x_sel=None, finalize=False):
        res = super().run_step(inp, x_sel=x_sel, finalize=False)
        if finalize:
            orc.fp8_append_block(self.sh, self.kv.page_table, self.kv_len, self.k_codes, self.v_codes, self.k_scale,
                                 self.v_scale, inp.k_blk, inp.v_blk)
            orc.fp8_dequantize_pages(self.sh, self.k_codes, self.v_codes, self.k_scale, self.v_scale, self.kv)
            orc.build_page_summaries(self.sh, self.kv)
            self.step[:] = 0
        return res


def delta_gap_ok(delta_row, m, rel=1e-3):
    """The m-th and (m+1)-th largest Delta are clearly separated, or exactly equal (then the index
    tie rule decides on both sides).  Otherwise fp rounding could flip the selection."""
    d = np.sort(np.asarray(delta_row))[::-1]
    if m <= 0 or m >= d.size:
        return True
    a, b = d[m - 1], d[m]
    return a == b or (a - b) > rel * max(abs(a), abs(b))


def tau_gap_ok(delta_row, m, tau, rel=1e-9):
    """The threshold rule's decision is clear of rounding: the cumulative Delta of the first m ranked
    tokens exceeds tau * total by a margin, and that of the first m - 1 stays below it by one."""
    d = np.sort(np.asarray(delta_row, np.float64))[::-1]
    total = d.sum()
    if total == 0.0:
        return m == 0
    cum = np.cumsum(d)
    thr = tau * total
    hi_ok = m == d.size or m == 0 or cum[m - 1] - thr > rel * total or cum[m - 1] == thr
    lo_ok = m <= 1 or thr - cum[m - 2] > rel * total
    return bool(hi_ok and lo_ok)
