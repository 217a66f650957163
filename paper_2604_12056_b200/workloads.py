"""Seeded synthetic inputs for the LoSA denoise-step attention path.

This module only draws numbers and lays them out (paged KV pool, page table, per-step Q / K_b / V_b
with a few freshly drawn "active" tokens and many slightly perturbed "stable" ones).  It contains
none of the method's arithmetic — no scores, no selection, no attention — so that the CUDA library
and the CPU oracle can both be fed the same bytes without sharing code.

The generators stand in for the workload the paper measures (a trained block-diffusion model on a
long-context QA set, Section 5.4): they keep its shapes and structure — long paged prefix, a block
of B queries, few tokens changing a lot between steps and most barely changing (Section 3.2), keys
clustered per page so that page-level selection is informative and per-query selections overlap
only partly (Section 3.1).

Element tensors are numpy `float32` arrays or `uint16` arrays holding bf16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np

BASE_SEED = 12056 * 1000


# ---------------------------------------------------------------- bf16 bit patterns (formatting)
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of float32 values to bf16 bit patterns (uint16)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) >> 16).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        r = np.where(nan, np.uint16(0x7FC0), r)
    return r


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def to_elem(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return f32_to_bf16_bits(x) if dtype == "bf16" else x


def elem_to_f32(x: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(x) if x.dtype == np.uint16 else x.astype(np.float32)


# ---------------------------------------------------------------- configurations
@dataclass(frozen=True)
class Config:
    name: str
    index: int                      # position in the benchmark's config list (1-based)
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int
    kv_lens: tuple                  # prefix tokens per sequence
    block_size: int
    steps: int                      # denoising steps per block
    topk: int                       # per-query budget in pages
    m_active: int                   # active tokens per step >= 1 (planted)
    dtype: str                      # "f32" | "bf16"
    clustered: bool                 # page-clustered keys / topic-structured queries
    heavy_frac: float = 0.0         # fraction of pages aligned with the block's common direction
    rho: float = 0.7                # weight of the block's common direction in a query
    tau: float = 0.7                # query norm / sqrt(d)
    n_blocks: int = 1               # consecutive blocks (each finalised block is appended)
    beta_active: bool = False       # draw m per step from Beta(2, 18) * B instead of m_active
    hidden_width: int = 0           # width of an extra hidden-state tensor (0 = none)

    @property
    def batch(self) -> int:
        return len(self.kv_lens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def max_pages_per_seq(self) -> int:
        g = self.page_size
        return max((L + self.n_blocks * self.block_size + g - 1) // g for L in self.kv_lens)

    @property
    def sm_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


def active_count(frac: float, block: int) -> int:
    """m = clamp(round-half-up(frac * B), 1, B)."""
    return int(min(block, max(1, int(np.floor(frac * block + 0.5)))))


def config(name: str, **kw) -> Config:
    """The five benchmark configurations (c1 .. c5), the paper-shaped p1 / p2, and reduced variants for tests."""
    qwen = dict(n_q_heads=32, n_kv_heads=8, head_dim=128)
    table = {
        # tiny fp32 single layer: 64 pages of 16, block 16, 4 steps, 4 planted tokens, k = 8
        "c1": Config("c1", 1, 4, 1, 64, 16, (1024,), 16, 4, 8, 4, "f32", False, hidden_width=256),
        # Qwen3-8B-shaped layer, 8K prefix, pages of 32, block 32, 8 steps, ~10% active, k = 32
        "c2": Config("c2", 2, page_size=32, kv_lens=(8192,), block_size=32, steps=8, topk=32,
                     m_active=active_count(0.10, 32), dtype="bf16", clustered=True, **qwen),
        # ragged long-context batch 16K/24K/32K/32K, k = 64, active fraction swept by the caller
        "c3": Config("c3", 3, page_size=32, kv_lens=(16384, 24576, 32768, 32768), block_size=32,
                     steps=8, topk=64, m_active=active_count(0.10, 32), dtype="bf16",
                     clustered=True, **qwen),
        # 128K prefix, pages of 64, block 64, 16 steps, 8% active, 5% heavy-hitter pages
        "c4": Config("c4", 4, page_size=64, kv_lens=(131072,), block_size=64, steps=16, topk=64,
                     m_active=active_count(0.08, 64), dtype="bf16", clustered=True,
                     heavy_frac=0.05, rho=0.5, **qwen),
        # one layer of the multi-layer loop: batch 8 x 32K, 4 blocks of 8 steps, Beta(2,18) active
        "c5": Config("c5", 5, page_size=32, kv_lens=(32768,) * 8, block_size=32, steps=8, topk=64,
                     m_active=active_count(0.10, 32), dtype="bf16", clustered=True, n_blocks=4,
                     beta_active=True, **qwen),
        # the shapes of the paper's latency study (Section 5.4), batch 1, five active tokens per step,
        # budget 512 tokens = 16 pages by default: p1 = 64K context / block 16, p2 = 32K context / block 32
        "p1": Config("p1", 6, page_size=32, kv_lens=(65536,), block_size=16, steps=8, topk=16,
                     m_active=5, dtype="bf16", clustered=True, **qwen),
        "p2": Config("p2", 7, page_size=32, kv_lens=(32768,), block_size=32, steps=8, topk=16,
                     m_active=5, dtype="bf16", clustered=True, **qwen),
    }
    return replace(table[name], **kw)


def seed_for(cfg: Config, replica: int = 0, layer: int = 0) -> int:
    return BASE_SEED + 100 * cfg.index + 10 * replica + layer


# ---------------------------------------------------------------- per-step inputs
@dataclass
class StepInputs:
    q: np.ndarray                 # [N, B, H_q, d]
    k_blk: np.ndarray             # [N, B, H_kv, d]
    v_blk: np.ndarray             # [N, B, H_kv, d]
    hidden: Optional[np.ndarray]  # [N, B, hidden_width] or None
    planted: List[np.ndarray]     # per sequence: sorted token ids that were redrawn (step >= 1)
    frozen: List[int]             # per sequence: one stable token left bit-identical (-1 if none)
    m_per_seq: np.ndarray         # [N] int32 (B at step 0)


def _unit(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


@dataclass
class Workload:
    """A paged prefix pool plus the per-step block inputs of `cfg.n_blocks` blocks."""
    cfg: Config
    replica: int = 0
    layer: int = 0
    pad_nan: bool = True          # fill the unused tail of a partial last page with NaN
    k_pages: np.ndarray = field(init=False, repr=False)
    v_pages: np.ndarray = field(init=False, repr=False)
    page_table: np.ndarray = field(init=False, repr=False)
    kv_len: np.ndarray = field(init=False, repr=False)

    def __post_init__(self):
        c = self.cfg
        self.rng = np.random.Generator(np.random.PCG64(seed_for(c, self.replica, self.layer)))
        N, Hkv, g, d = c.batch, c.n_kv_heads, c.page_size, c.head_dim
        Pmax = c.max_pages_per_seq
        self.n_phys = N * Pmax
        perm = self.rng.permutation(self.n_phys).astype(np.int32)
        self.page_table = np.ascontiguousarray(perm.reshape(N, Pmax))
        self.kv_len = np.asarray(c.kv_lens, np.int32).copy()
        e = np.uint16 if c.dtype == "bf16" else np.float32
        self.k_pages = np.zeros((self.n_phys, Hkv, g, d), e)
        self.v_pages = np.zeros((self.n_phys, Hkv, g, d), e)
        self.page_means = []      # per sequence [P, H_kv, d] unit vectors (clustered only)
        self.common_dir = []      # per sequence [H_kv, d]
        for s in range(N):
            self._fill_prefix(s)
        self._cur = None

    # -- prefix ---------------------------------------------------------------------------------
    def _fill_prefix(self, s: int):
        c, rng = self.cfg, self.rng
        Hkv, g, d = c.n_kv_heads, c.page_size, c.head_dim
        L = int(self.kv_len[s])
        P = (L + g - 1) // g
        if P == 0:
            self.page_means.append(np.zeros((0, Hkv, d), np.float32))
            self.common_dir.append(_unit(rng.standard_normal((Hkv, d), dtype=np.float32)))
            return
        if c.clustered:
            u = _unit(rng.standard_normal((P, Hkv, d), dtype=np.float32))
            pick = rng.integers(0, P, size=(Hkv, 16))
            cdir = _unit(np.stack([u[pick[h], h].sum(0) for h in range(Hkv)]))
            if c.heavy_frac > 0:
                nh = int(round(c.heavy_frac * P))
                heavy = rng.choice(P, size=nh, replace=False)
                o = rng.standard_normal((nh, Hkv, d), dtype=np.float32)
                o = _unit(o - (o * cdir[None]).sum(-1, keepdims=True) * cdir[None])
                u[heavy] = 0.8 * cdir[None] + 0.6 * o
            self.page_means.append(u)
            self.common_dir.append(cdir)
        phys = self.page_table[s, :P]
        chunk = max(1, (1 << 24) // (Hkv * g * d))
        for p0 in range(0, P, chunk):
            p1 = min(P, p0 + chunk)
            noise = rng.standard_normal((p1 - p0, Hkv, g, d), dtype=np.float32)
            if c.clustered:
                kk = np.float32(np.sqrt(d)) * self.page_means[s][p0:p1, :, None, :] + np.float32(0.5) * noise
                vv = rng.standard_normal((p1 - p0, Hkv, g, d), dtype=np.float32)
            else:
                kk = noise / np.float32(np.sqrt(d))
                vv = rng.standard_normal((p1 - p0, Hkv, g, d), dtype=np.float32) / np.float32(np.sqrt(d))
            if p1 == P and L % g and self.pad_nan:
                kk[-1, :, L % g:, :] = np.nan
                vv[-1, :, L % g:, :] = np.nan
            self.k_pages[phys[p0:p1]] = to_elem(kk, c.dtype)
            self.v_pages[phys[p0:p1]] = to_elem(vv, c.dtype)

    # -- block inputs -----------------------------------------------------------------------------
    def _draw_q_rows(self, s: int, n: int) -> np.ndarray:
        """n fresh query rows [n, H_q, d] for sequence s."""
        c, rng = self.cfg, self.rng
        Hq, d, G = c.n_q_heads, c.head_dim, c.group
        if not c.clustered or self.page_means[s].shape[0] == 0:
            return rng.standard_normal((n, Hq, d), dtype=np.float32) / np.float32(np.sqrt(d))
        u = self.page_means[s]
        P = u.shape[0]
        pick = rng.integers(0, P, size=(n, Hq, 8))
        kh = np.arange(Hq) // G
        t = u[pick, kh[None, :, None]].sum(2)                          # [n, H_q, d]
        if P < 8:   # too few pages to make fresh draws differ: add a random direction
            t = _unit(t) + np.float32(0.5) * _unit(rng.standard_normal((n, Hq, d), dtype=np.float32))
        t = _unit(t)
        cd = self.common_dir[s][kh][None]                               # [1, H_q, d]
        mix = np.float32(c.rho) * cd + np.float32(np.sqrt(1 - c.rho ** 2)) * t
        return (np.float32(c.tau * np.sqrt(d)) * _unit(mix)).astype(np.float32)

    def _draw_kv_rows(self, s: int, n: int):
        c, rng = self.cfg, self.rng
        Hkv, d = c.n_kv_heads, c.head_dim
        if c.clustered:
            k = np.float32(np.sqrt(d)) * self._blk_mean[s][None] + np.float32(0.5) * rng.standard_normal((n, Hkv, d), dtype=np.float32)
            v = rng.standard_normal((n, Hkv, d), dtype=np.float32)
        else:
            k = rng.standard_normal((n, Hkv, d), dtype=np.float32) / np.float32(np.sqrt(d))
            v = rng.standard_normal((n, Hkv, d), dtype=np.float32) / np.float32(np.sqrt(d))
        return k, v

    def start_block(self) -> StepInputs:
        """Step 0 of a new block: everything freshly drawn."""
        c, rng = self.cfg, self.rng
        N, B = c.batch, c.block_size
        self._blk_mean = [_unit(rng.standard_normal((c.n_kv_heads, c.head_dim), dtype=np.float32)) for _ in range(N)]
        q = np.stack([self._draw_q_rows(s, B) for s in range(N)])
        kv = [self._draw_kv_rows(s, B) for s in range(N)]
        k = np.stack([a for a, _ in kv])
        v = np.stack([b for _, b in kv])
        h = (rng.standard_normal((N, B, c.hidden_width), dtype=np.float32) / np.float32(np.sqrt(c.head_dim))
             if c.hidden_width else None)
        self._cur = (q, k, v, h)
        return self._pack([np.arange(B)] * N, [-1] * N, np.full(N, B, np.int32))

    def next_step(self, m: Optional[int] = None) -> StepInputs:
        """Step >= 1: m seeded tokens per sequence are redrawn, one stable token stays
        bit-identical, the others get additive N(0, 1e-3) noise."""
        c, rng = self.cfg, self.rng
        N, B = c.batch, c.block_size
        if m is None:
            m = c.m_active
            if c.beta_active:
                m = int(min(B, max(1, int(np.floor(rng.beta(2.0, 18.0) * B + 0.5)))))
        q, k, v, h = (None if a is None else elem_to_f32(to_elem(a, c.dtype)).copy() for a in self._cur)
        planted, frozen = [], []
        for s in range(N):
            act = np.sort(rng.choice(B, size=m, replace=False))
            stable = np.setdiff1d(np.arange(B), act)
            fz = int(rng.choice(stable)) if stable.size else -1
            noisy = stable[stable != fz]
            q[s, act] = self._draw_q_rows(s, m)
            kk, vv = self._draw_kv_rows(s, m)
            k[s, act], v[s, act] = kk, vv
            sd = np.float32(1e-3)
            q[s, noisy] += sd * rng.standard_normal((noisy.size,) + q.shape[2:], dtype=np.float32)
            k[s, noisy] += sd * rng.standard_normal((noisy.size,) + k.shape[2:], dtype=np.float32)
            v[s, noisy] += sd * rng.standard_normal((noisy.size,) + v.shape[2:], dtype=np.float32)
            if h is not None:
                h[s, act] = rng.standard_normal((m, c.hidden_width), dtype=np.float32) / np.float32(np.sqrt(c.head_dim))
                h[s, noisy] += sd * rng.standard_normal((noisy.size, c.hidden_width), dtype=np.float32)
            planted.append(act)
            frozen.append(fz)
        self._cur = (q, k, v, h)
        return self._pack(planted, frozen, np.full(N, m, np.int32))

    def _pack(self, planted, frozen, m_per_seq) -> StepInputs:
        c = self.cfg
        q, k, v, h = self._cur
        return StepInputs(to_elem(q, c.dtype), to_elem(k, c.dtype), to_elem(v, c.dtype),
                          None if h is None else to_elem(h, c.dtype), planted, frozen, m_per_seq)

    def block_steps(self, m: Optional[int] = None) -> List[StepInputs]:
        """All `cfg.steps` steps of one block."""
        out = [self.start_block()]
        for _ in range(1, self.cfg.steps):
            out.append(self.next_step(m))
        return out

    # -- bookkeeping ------------------------------------------------------------------------------
    def pool_bytes(self) -> int:
        return self.k_pages.nbytes + self.v_pages.nbytes


# ---------------------------------------------------------------- device-side generation (torch)
class DeviceWorkload:
    """The same recipe as `Workload`, drawn with torch on a CUDA device.

    Used where host generation would take minutes (the 36-layer configuration: about 1 GiB of K/V
    per layer).  Tensors live on the device (bf16 / fp32 / int32); `host_copy()` returns numpy
    arrays in the formats `Workload` uses, so that a CPU checker can be fed the same bytes.  The
    number of active tokens per step is drawn on the host from a seed that does not depend on the
    layer, so all layers of a model share it."""

    def __init__(self, cfg: Config, replica: int = 0, layer: int = 0, device="cuda"):
        import torch
        self.torch = torch
        self.cfg, self.replica, self.layer, self.device = cfg, replica, layer, device
        self.gen = torch.Generator(device=device)
        self.gen.manual_seed(seed_for(cfg, replica, layer))
        self.m_rng = np.random.Generator(np.random.PCG64(seed_for(cfg, replica, 0) + 7))
        self.dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        N, Hkv, g, d = cfg.batch, cfg.n_kv_heads, cfg.page_size, cfg.head_dim
        Pmax = cfg.max_pages_per_seq
        self.n_phys = N * Pmax
        self.page_table = torch.randperm(self.n_phys, generator=self.gen, device=device).to(torch.int32).reshape(N, Pmax).contiguous()
        self.kv_len = torch.tensor(cfg.kv_lens, dtype=torch.int32, device=device)
        self.k_pages = torch.zeros((self.n_phys, Hkv, g, d), dtype=self.dt, device=device)
        self.v_pages = torch.zeros((self.n_phys, Hkv, g, d), dtype=self.dt, device=device)
        self.page_means, self.common_dir = [], []
        for s in range(N):
            self._fill_prefix(s)
        self._cur = None

    def _randn(self, *shape):
        return self.torch.randn(*shape, generator=self.gen, device=self.device, dtype=self.torch.float32)

    def _unit(self, x):
        return x / x.norm(dim=-1, keepdim=True)

    def _fill_prefix(self, s):
        torch, c = self.torch, self.cfg
        Hkv, g, d = c.n_kv_heads, c.page_size, c.head_dim
        L = int(c.kv_lens[s])
        P = (L + g - 1) // g
        if P == 0:
            self.page_means.append(torch.zeros((0, Hkv, d), device=self.device))
            self.common_dir.append(self._unit(self._randn(Hkv, d)))
            return
        rt_d = float(np.sqrt(d))
        if c.clustered:
            u = self._unit(self._randn(P, Hkv, d))
            pick = torch.randint(0, P, (Hkv, 16), generator=self.gen, device=self.device)
            cdir = self._unit(torch.stack([u[pick[h], h].sum(0) for h in range(Hkv)]))
            if c.heavy_frac > 0:
                nh = int(round(c.heavy_frac * P))
                heavy = torch.randperm(P, generator=self.gen, device=self.device)[:nh]
                o = self._randn(nh, Hkv, d)
                o = self._unit(o - (o * cdir[None]).sum(-1, keepdim=True) * cdir[None])
                u[heavy] = 0.8 * cdir[None] + 0.6 * o
            self.page_means.append(u)
            self.common_dir.append(cdir)
        phys = self.page_table[s, :P].long()
        chunk = max(1, (1 << 26) // (Hkv * g * d))
        for p0 in range(0, P, chunk):
            p1 = min(P, p0 + chunk)
            noise = self._randn(p1 - p0, Hkv, g, d)
            if c.clustered:
                kk = rt_d * self.page_means[s][p0:p1, :, None, :] + 0.5 * noise
                vv = self._randn(p1 - p0, Hkv, g, d)
            else:
                kk = noise / rt_d
                vv = self._randn(p1 - p0, Hkv, g, d) / rt_d
            if p1 == P and L % g:
                kk[-1, :, L % g:, :] = float("nan")
                vv[-1, :, L % g:, :] = float("nan")
            self.k_pages[phys[p0:p1]] = kk.to(self.dt)
            self.v_pages[phys[p0:p1]] = vv.to(self.dt)

    def _draw_q_rows(self, s, n):
        torch, c = self.torch, self.cfg
        Hq, d, G = c.n_q_heads, c.head_dim, c.group
        if not c.clustered or self.page_means[s].shape[0] == 0:
            return self._randn(n, Hq, d) / float(np.sqrt(d))
        u = self.page_means[s]
        P = u.shape[0]
        pick = torch.randint(0, P, (n, Hq, 8), generator=self.gen, device=self.device)
        kh = (torch.arange(Hq, device=self.device) // G)
        t = u[pick, kh[None, :, None]].sum(2)
        if P < 8:
            t = self._unit(t) + 0.5 * self._unit(self._randn(n, Hq, d))
        t = self._unit(t)
        cd = self.common_dir[s][kh][None]
        mix = c.rho * cd + float(np.sqrt(1 - c.rho ** 2)) * t
        return float(c.tau * np.sqrt(d)) * self._unit(mix)

    def _draw_kv_rows(self, s, n):
        c = self.cfg
        Hkv, d = c.n_kv_heads, c.head_dim
        if c.clustered:
            k = float(np.sqrt(d)) * self._blk_mean[s][None] + 0.5 * self._randn(n, Hkv, d)
            v = self._randn(n, Hkv, d)
        else:
            k = self._randn(n, Hkv, d) / float(np.sqrt(d))
            v = self._randn(n, Hkv, d) / float(np.sqrt(d))
        return k, v

    def start_block(self):
        torch, c = self.torch, self.cfg
        N, B = c.batch, c.block_size
        self._blk_mean = [self._unit(self._randn(c.n_kv_heads, c.head_dim)) for _ in range(N)]
        q = torch.stack([self._draw_q_rows(s, B) for s in range(N)])
        kv = [self._draw_kv_rows(s, B) for s in range(N)]
        k = torch.stack([a for a, _ in kv])
        v = torch.stack([b for _, b in kv])
        self._cur = tuple(x.to(self.dt).float() for x in (q, k, v))
        return self._pack([np.arange(B)] * N, np.full(N, B, np.int32))

    def draw_m(self) -> int:
        c = self.cfg
        if c.beta_active:
            return int(min(c.block_size, max(1, int(np.floor(self.m_rng.beta(2.0, 18.0) * c.block_size + 0.5)))))
        return c.m_active

    def next_step(self, m: Optional[int] = None):
        torch, c = self.torch, self.cfg
        N, B = c.batch, c.block_size
        if m is None:
            m = self.draw_m()
        q, k, v = (x.clone() for x in self._cur)
        planted = []
        for s in range(N):
            perm = torch.randperm(B, generator=self.gen, device=self.device)
            act = perm[:m].sort().values
            noisy = perm[m:]
            q[s, act] = self._draw_q_rows(s, m)
            kk, vv = self._draw_kv_rows(s, m)
            k[s, act], v[s, act] = kk, vv
            q[s, noisy] += 1e-3 * self._randn(noisy.numel(), *q.shape[2:])
            k[s, noisy] += 1e-3 * self._randn(noisy.numel(), *k.shape[2:])
            v[s, noisy] += 1e-3 * self._randn(noisy.numel(), *v.shape[2:])
            planted.append(act.cpu().numpy())
        self._cur = tuple(x.to(self.dt).float() for x in (q, k, v))
        return self._pack(planted, np.full(N, m, np.int32))

    def _pack(self, planted, m_per_seq):
        q, k, v = (x.to(self.dt).contiguous() for x in self._cur)
        return DeviceStepInputs(q, k, v, planted, self.torch.from_numpy(m_per_seq).to(self.device))

    def host_copy(self):
        """numpy view of the pool for a CPU checker (bf16 as uint16 bit patterns)."""
        import types
        def np_of(t):
            t = t.detach().cpu()
            return t.view(self.torch.int16).numpy().view(np.uint16) if t.dtype == self.torch.bfloat16 else t.numpy()
        return types.SimpleNamespace(cfg=self.cfg, k_pages=np_of(self.k_pages), v_pages=np_of(self.v_pages),
                                     page_table=np_of(self.page_table), kv_len=np_of(self.kv_len), n_phys=self.n_phys)


@dataclass
class DeviceStepInputs:
    q: object
    k_blk: object
    v_blk: object
    planted: List[np.ndarray]
    m_per_seq: object

    def host_copy(self) -> StepInputs:
        import torch
        def np_of(t):
            t = t.detach().cpu()
            return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()
        return StepInputs(np_of(self.q), np_of(self.k_blk), np_of(self.v_blk), None, self.planted,
                          [-1] * len(self.planted), np_of(self.m_per_seq).astype(np.int32))
