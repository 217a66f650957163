#!/usr/bin/env python
"""Benchmark of the LoSA denoise-step attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c3]

One "step" is one layer-step: stages 1-6 of include/losa.h for one attention layer and one
denoising step, issued through the whole-step entry point losa_denoise_step.  The K timed steps walk
whole denoising blocks in model order (block, denoising step, layer) from a block boundary, over
min(layers, ceil(K / T)) layers: step 0 of a block is the dense first step, the other T-1 are LoSA
steps, so K steps hold ceil(K / T) dense ones and their mean is the block average when T divides K
(see schedule()).  Before them, whole blocks of the same layers run untimed (at least W steps).
Prints ONE JSON line and exits non-zero if no LoSA step was measured.

Timing: with one layer, the layer-step is captured once in a CUDA graph and replayed; each step is
bracketed by CUDA events on the launching stream; between steps, outside the timed region, the L2
is flushed by writing a 256 MiB buffer and then reading a second one (the read pass makes the cache
write its dirty lines back, so that write-back traffic of the flush itself does not land in the
timed step).  With several layers (the default), one denoising step of the timed layers - their
steps in order, each on its own ~1 GiB KV pool, so nothing a step reads is left in L2 - is one CUDA
graph; one event pair brackets each replay and a layer-step counts as 1/n of it.
The time of K steps is the sum of the event intervals; with several
GPUs every rank runs its own replica of the workload (weak scaling, no data-path collective) and
the maximum over ranks is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_12056_b200 import workloads as wl  # noqa: E402

METRIC = "denoise-step attention us/layer"
UNIT = "us/layer-step"
L2_FLUSH_BYTES = 256 << 20
# DRAM traffic of the stage-4 main kernel per listed (page, KV head) slice, from the ncu capture in
# profiles/attn_tc5_kernel_c5.txt: the dense launch there moved dram__bytes_read.sum +
# dram__bytes_write.sum = 1,077.27 + 5.16 MB for its 65,536 slices (16,384 of the 16,516 bytes per slice
# are the slice's K and V).  Traffic grows in proportion to the slices, so a launch's traffic is reported
# as slices x this figure; LoSA launches add the partial records they write (3.4-4.7 MB of DRAM writes
# in the three LoSA launches of that capture).  Pages of 32 tokens, head dim 128, bf16; other page sizes
# scale by the slice size (pages of 64 with two row groups per KV head, workload c4: 537.6 MB read for
# 16,384 slices of 32,768 bytes on the dense step, 1.001 of the slices' bytes: the second row group's
# pass over the pages is served by the L2, see profiles/attn_tc5_kernel_c4.txt).
NCU_BYTES_PER_SLICE = {"losa": 1082.43e6 / 65536, "dense": 1082.43e6 / 65536}
NCU_FIXED_BYTES = {"losa": 4.2e6, "dense": 0.0}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed layer-steps (default: 4 blocks of all layers)")
    ap.add_argument("--warmup", type=int, default=0, help="untimed layer-steps (default: 1 block of all layers)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5", "p1", "p2"])
    ap.add_argument("--topk", type=int, default=0, help="override the page budget per query (pages)")
    ap.add_argument("--pooled", action="store_true",
                    help="selector variant: one page list per (token, KV head) instead of one per query head")
    ap.add_argument("--layers", type=int, default=0, help="attention layers (default: 36 for c5, else 1)")
    ap.add_argument("--active-frac", type=float, default=None, help="override the active fraction")
    ap.add_argument("--selector", default="exact", choices=["exact", "mma"],
                    help="mma: stage 2 takes its page scores from a tensor-core GEMM; lists valid under the relaxed rule")
    ap.add_argument("--state-dtype", default="f32", choices=["f32", "bf16"],
                    help="bf16: the cached prefix output of the per-block state is stored rounded to bf16")
    ap.add_argument("--kv-dtype", default="native", choices=["native", "fp8"],
                    help="fp8: the K/V pages are stored as E4M3 bytes with one power-of-two scale per (page, KV head)")
    ap.add_argument("--no-extras", action="store_true", help="skip baselines, stage breakdown, cpu baseline")
    return ap.parse_args()


def make_config(args):
    cfg = wl.config(args.workload)
    if args.topk > 0:
        cfg = wl.config(args.workload, topk=args.topk)
    if args.active_frac is not None:
        cfg = wl.config(args.workload, m_active=wl.active_count(args.active_frac, cfg.block_size),
                        n_blocks=cfg.n_blocks, beta_active=False, topk=cfg.topk)
    return cfg


def workload_name(cfg, layers=1):
    lens = "/".join(f"{L // 1024}K" for L in cfg.kv_lens)
    if len(set(cfg.kv_lens)) == 1:
        lens = f"{cfg.kv_lens[0] // 1024}K"
    act = "Beta(2,18)*B active tokens/step" if cfg.beta_active else f"{cfg.m_active} active tokens/step"
    return (f"{cfg.name}: {layers} layer(s), batch {cfg.batch}, prefix {lens} tokens, pages of {cfg.page_size}, "
            f"{cfg.n_q_heads}/{cfg.n_kv_heads} heads x {cfg.head_dim}, block {cfg.block_size}, "
            f"{cfg.steps} steps/block, {act}, top-{cfg.topk} pages, {cfg.dtype}")


# ------------------------------------------------------------------------------- clocks sampling
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (every ~2 ms) while the timed region runs."""

    def __init__(self, index):
        self.index, self.rows, self._stop, self._thr, self.max_mhz = index, [], False, None, None

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = int(visible.split(",")[self.index]) if visible and visible.split(",")[self.index].isdigit() else self.index
            h = nv.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
        except Exception:
            return

        def loop():
            while not self._stop:
                try:
                    self.rows.append((float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                      int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))))
                except Exception:
                    try:
                        self.rows.append((float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                          int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))))
                    except Exception:
                        pass
                time.sleep(0.002)
        self._thr = threading.Thread(target=loop, daemon=True)
        self._thr.start()

    def stop(self):
        self._stop = True
        if self._thr:
            self._thr.join(timeout=2)
        bits = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}
        sm = sorted(r[0] for r in self.rows)
        reasons = sorted(n for n, b in bits.items() if any(r[1] & b for r in self.rows))
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sm)}


# ------------------------------------------------------------------------------- byte accounting
def stage4_bytes(cfg, up, uc, na, kv_len, fp8=False):
    """Algorithmic bytes of one stage-4 launch: K and V of the valid tokens of every listed page,
    the active queries, the union list and page-table entries read, the state rows written (FP8
    pages: one byte per K / V element plus the two scales of every listed page)."""
    e = 2 if cfg.dtype == "bf16" else 4
    ekv = 1 if fp8 else e
    g, d = cfg.page_size, cfg.head_dim
    total = 0
    for s in range(cfg.batch):
        if na[s] == 0:
            continue
        P = (int(kv_len[s]) + g - 1) // g
        tail = int(kv_len[s]) - (P - 1) * g if P else 0
        for kh in range(cfg.n_kv_heads):
            n = int(uc[s, kh])
            toks = n * g
            if n and up[s, kh, n - 1] == P - 1:    # lists ascend: only the last entry can be the partial page
                toks -= g - tail
            total += 2 * toks * d * ekv + 8 * n + (8 * n if fp8 else 0)
        total += int(na[s]) * cfg.n_q_heads * (d * e + (d + 1) * 4)
    return total


def pages_read(uc):
    return int(np.asarray(uc).sum())


# ------------------------------------------------------------------------------- oracle timing
def oracle_block_time(cfg, w, steps_inputs, sample_tokens=2):
    """Seconds per layer-step of the oracle as it stands, averaged over one block: LoSA steps in
    full; the dense first step's prefix attention on `sample_tokens` of the B block tokens, scaled
    by B / sample_tokens (its cost is linear in the number of query tokens)."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import OracleLayer
    from oracle import oracle as orc
    lay = OracleLayer(w, "losa")
    sh = lay.sh
    inp0 = steps_inputs[0]
    N, B = cfg.batch, cfg.block_size
    # dense first step, sampled
    t0 = time.perf_counter()
    act, na, _ = orc.select_active(sh, inp0.q, lay.q_prev, inp0.m_per_seq, lay.step)
    up, uc = orc.page_union(sh, lay.topk, act, na, cfg.topk, lay.kv_len, lay.step)
    t_idx = time.perf_counter() - t0
    act_s = np.full((N, B), -1, np.int32)
    act_s[:, :sample_tokens] = np.arange(sample_tokens)
    na_s = np.full(N, sample_tokens, np.int32)
    t0 = time.perf_counter()
    orc.sparse_prefix_attn(sh, inp0.q, lay.kv, act_s, na_s, up, uc, lay.o_p, lay.lse_p)
    t_attn = (time.perf_counter() - t0) * (B / sample_tokens)
    t0 = time.perf_counter()
    orc.block_attn_merge(sh, inp0.q, inp0.k_blk, inp0.v_blk, lay.o_p, lay.lse_p)
    orc.update_prefix_cache(sh, lay.kv, lay.q_prev, lay.step, inp0.q, inp0.k_blk, inp0.v_blk, False)
    t_dense = t_idx + t_attn + (time.perf_counter() - t0)
    # one LoSA step in full
    t0 = time.perf_counter()
    lay.run_step(steps_inputs[1])
    t_sparse = time.perf_counter() - t0
    T = cfg.steps
    return (t_dense + (T - 1) * t_sparse) / T, t_dense, t_sparse, orc.num_threads()


def run_reference(args, cfg):
    """--impl reference: the CPU oracle, as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    orc.build()
    w = wl.Workload(cfg)
    steps_inputs = w.block_steps()
    times, t_start, n_warm = [], time.perf_counter(), 0
    while True:
        per_step, t_dense, t_sparse, cores = oracle_block_time(cfg, w, steps_inputs)
        wall = time.perf_counter() - t_start
        if n_warm < args.warmup and wall < 45:
            n_warm += 1                       # untimed warm-up sample
            continue
        times.append(per_step)
        if len(times) >= args.steps or wall > 200:      # keep the whole run within a few minutes
            break
    timed = times
    us = float(np.mean(timed)) * 1e6
    sample = (f"per step: one full LoSA layer-step and a dense first step whose prefix attention runs on 2 of "
              f"{cfg.block_size} block tokens (x{cfg.block_size // 2}), averaged over a block of {cfg.steps}; "
              f"{len(timed)} such samples")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(timed), "warmup": n_warm, "ms_per_step": us / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, args.layers if args.layers else (36 if cfg.name == "c5" else 1)),
                   "note": "the layers differ only in their seeds; the oracle is timed on layer 0"},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------- GPU arm
class LayerRun:
    """One attention layer of the workload on the device: its own seeded pool, LoSA cache, static
    input buffers and two CUDA graphs (the whole-step call; block finalisation)."""

    def __init__(self, cfg, rank, layer, dev, pooled=False, fp8=False, state_bf16=False, mma=False):
        import torch
        from paper_2604_12056_b200.layer import LosaLayer
        self.torch, self.cfg = torch, cfg
        self.w = wl.DeviceWorkload(cfg, replica=rank, layer=layer, device=dev)
        self.layer = LosaLayer(cfg, self.w.k_pages, self.w.v_pages, self.w.page_table, self.w.kv_len, "losa", dev,
                               pooled=pooled, fp8_kv=fp8, state_bf16=state_bf16, mma_selector=mma)
        self.pool_mib = self.w.k_pages.numel() * (2 if fp8 else 4) / 2 ** 20
        if fp8:                                # the library has quantised the pools: release the bf16 copies
            torch.cuda.synchronize()
            self.w.k_pages = self.w.v_pages = None
            self.layer.k_pages = self.layer.v_pages = self.layer.kv_native = None
        self.inputs = {}                       # block -> list of DeviceStepInputs (current and previous block)
        self.next_block = 0
        first = self.block_inputs(0)[0]
        self.q_s, self.k_s, self.v_s, self.m_s = (torch.empty_like(t) for t in (first.q, first.k_blk, first.v_blk, first.m_per_seq))
        self.graph = self.graph_fin = None

    def block_inputs(self, b):
        """Inputs of block b (generated in block order; every layer draws the same active counts)."""
        assert b >= self.next_block - 2, "blocks are generated in order; only the last two are kept"
        while self.next_block <= b:
            nb = self.next_block
            self.inputs[nb] = [self.w.start_block()] + [self.w.next_step() for _ in range(self.cfg.steps - 1)]
            self.next_block = nb + 1
            for old in [k for k in self.inputs if k < nb - 1]:
                del self.inputs[old]
        return self.inputs[b]

    def load(self, b, t):
        i = self.block_inputs(b)[t]
        self.q_s.copy_(i.q); self.k_s.copy_(i.k_blk); self.v_s.copy_(i.v_blk); self.m_s.copy_(i.m_per_seq)

    def capture(self):
        torch = self.torch
        self.load(0, 0)
        self.layer.run_step_fused(self.q_s, self.k_s, self.v_s, self.m_s)      # un-captured first call
        torch.cuda.synchronize()
        self.layer.step.zero_()
        n0 = self.layer.ctx.launch_count()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.layer.run_step_fused(self.q_s, self.k_s, self.v_s, self.m_s)
        n1 = self.layer.ctx.launch_count()
        self.graph_fin = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_fin):
            self.layer.finalize_block(self.k_s, self.v_s)
        return n1 - n0, self.layer.ctx.launch_count() - n1


def schedule(K, T, L):
    """The walk of K layer-steps: model order (block, denoising step, layer) over
    L_eff = min(L, ceil(K / T)) layers, starting at a block boundary.  Returns L_eff and the sweeps
    [(block, t, n_layers)]: a sweep is one denoising step t of layers 0 .. n_layers-1 (only the last
    sweep can be partial).  The first sweep of a block is the dense first step, so K layer-steps
    hold ceil(K / T) dense ones (as long as K <= T * L, else the walk runs on into further blocks)
    and the mean over the walk equals the block average (1 dense + T-1 LoSA) when T divides K."""
    L_eff = max(1, min(L, -(-K // T)))
    sweeps, k = [], 0
    while k < K:
        n = min(L_eff, K - k)
        sw = k // L_eff
        sweeps.append((sw // T, sw % T, n))
        k += n
    return L_eff, sweeps


def run_ours(args, cfg0):
    import torch
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200 import build as build_mod
    from paper_2604_12056_b200 import dist as D
    from paper_2604_12056_b200.layer import to_host

    local = D.env_rank()[2]
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rank, world, local = D.init("nccl", dev)
    if not os.path.exists(B.LIB_PATH):
        if local == 0:
            build_mod.build()
        D.barrier()

    L_model = args.layers if args.layers else (36 if cfg0.name == "c5" else 1)
    T = cfg0.steps
    K = args.steps
    L, sweeps = schedule(K, T, L_model)
    n_dense_sched = sum(n for _, t, n in sweeps if t == 0)
    if n_dense_sched == K:
        sys.exit(f"bench.py: --steps {K} holds no LoSA step (a block has {T} steps, the first one dense); "
                 "the metric is defined on the sparse steps")
    per_block = T * L
    blocks_region = sweeps[-1][0] + 1                          # blocks one pass over the schedule touches
    warm_blocks = max(1, -(-args.warmup // per_block))         # whole untimed blocks: at least W layer-steps
    total_blocks = warm_blocks + 4 * blocks_region + 3
    cfg = wl.config(cfg0.name, n_blocks=total_blocks, m_active=cfg0.m_active, beta_active=cfg0.beta_active, topk=cfg0.topk)
    fp8 = args.kv_dtype == "fp8"
    runs = [LayerRun(cfg, D.replica_of(rank), l, dev, pooled=args.pooled, fp8=fp8, state_bf16=args.state_dtype == "bf16",
                     mma=args.selector == "mma") for l in range(L)]
    launches_step = launches_fin = 0
    for r in runs:
        launches_step, launches_fin = r.capture()
    flush_w = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)   # fp32: sum() reads it in place
    use_flush = L == 1            # with several layers, consecutive steps read different ~1 GiB pools

    def flush(v, force=False):
        """Evicts the L2 (write > L2, then read > L2 so that no dirty lines are left behind)."""
        if use_flush or force:
            flush_w.fill_(v & 0xff)
            flush_r.sum()

    state = {"launches": 0}

    # With several layers, one sweep (one denoising step of all timed layers, in order) is one CUDA
    # graph, as a serving engine would capture it; the last step of a block also finalises each
    # layer's block.  One event pair per sweep; a layer-step counts as 1/n of its sweep.
    model_graphs = None
    if L > 1:
        model_graphs = []
        for with_fin in (False, True):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for r in runs:
                    r.layer.run_step_fused(r.q_s, r.k_s, r.v_s, r.m_s)
                    if with_fin:
                        r.layer.finalize_block(r.k_s, r.v_s)
            model_graphs.append(g)
    for r in runs:
        r.layer.step.zero_()

    def timed_pass(block0, sw_list, record=None):
        """Replays the sweeps of `sw_list` (block numbers relative to block0).  Returns one
        (t, n_layers, milliseconds) per sweep.  Nothing is read back inside the loop (the union
        sizes go to a device log), so the host runs ahead and the sweeps execute back to back."""
        evs = []
        log = torch.zeros((len(sw_list), L), dtype=torch.int64, device=dev) if record is not None else None
        for j, (b, t, n) in enumerate(sw_list):
            for r in runs[:n]:
                r.load(block0 + b, t)
            flush(j)
            fin = t == T - 1
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if model_graphs is not None and n == L:
                model_graphs[1 if fin else 0].replay()
            else:
                for r in runs[:n]:
                    r.graph.replay()
                    if fin:
                        r.graph_fin.replay()                   # the block is finalised: append K_b, V_b
            e1.record()
            evs.append((e0, e1))
            state["launches"] += n * (launches_step + (launches_fin if fin else 0))
            if log is not None:
                for l, r in enumerate(runs[:n]):
                    log[j, l] = r.layer.union_count.sum()      # device-side, outside the event pair
        torch.cuda.synchronize()
        out = [(t, n, a.elapsed_time(b2)) for (_, t, n), (a, b2) in zip(sw_list, evs)]
        if record is not None:
            host_log = log.cpu().tolist()
            for j, (_, t, n) in enumerate(sw_list):
                record.extend((t, int(x)) for x in host_log[j][:n])
        return out

    # untimed: whole blocks from their dense first step on (state set-up and warm-up)
    warm_sweeps = [(b, t, L) for b in range(warm_blocks) for t in range(T)]
    timed_pass(0, warm_sweeps)
    D.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    pages = []
    state["launches"] = 0
    res = timed_pass(warm_blocks, sweeps, pages)
    torch.cuda.synchronize()
    D.barrier()
    clocks = sampler.stop()
    for r in runs:
        assert r.layer.ctx.poll_status() == 0
    total_ms = D.max_over_ranks(float(sum(ms for _, _, ms in res)), dev)
    ms_per_step = total_ms / K
    sparse_ms = [ms / n for t, n, ms in res if t != 0]
    dense_ms = [ms / n for t, n, ms in res if t == 0]
    n_dense = sum(n for t, n, _ in res if t == 0)

    result = {
        "metric": METRIC, "value": ms_per_step * 1e3, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": workload_name(cfg0, L_model) + (", pooled selector (one page list per token and KV head)" if args.pooled else "")
                               + (", K/V pages stored as FP8 E4M3 with per-page scales" if fp8 else "")
                               + (", cached prefix output stored as bf16" if args.state_dtype == "bf16" else "")
                               + (", tensor-core page scores (relaxed list rule)" if args.selector == "mma" else ""),
                   "sequences_per_gpu": cfg.batch, "layers": L_model, "layers_timed": L,
                   "step": "one layer-step = stages 1-6 for one layer and one denoising step; steps run in model order "
                           "(block, denoising step, layer) from a block boundary; the last step of a block also appends the block to the cache",
                   "timed_mix": {"dense_first_steps": n_dense, "losa_steps": K - n_dense,
                                 "note": f"{K} layer-steps over {L} of the {L_model} layers: ceil(K / {T}) dense first steps and the rest LoSA "
                                         f"steps, so that the mean is the block average (1 dense + {T - 1} LoSA) when {T} divides K"},
                   "untimed_before": f"{warm_blocks} whole block(s) of the {L} timed layers ({warm_blocks * per_block} layer-steps >= the {args.warmup} requested)",
                   "launch": ("CUDA graph replay of one denoising step of the timed layers (losa_denoise_step per layer, in order), "
                              "one event pair per denoising step" if L > 1 else
                              "CUDA graph replay of losa_denoise_step (stages 1-6 in one call), one graph per layer-step"),
                   "l2": ("flushed between steps, outside the timed region: 256 MiB write, then 256 MiB read so no dirty "
                          "lines remain") if use_flush else
                         ("inputs larger than L2: consecutive layer-steps read different per-layer KV pools "
                          f"({runs[0].pool_mib:.0f} MiB each), no flush")},
        "clocks": clocks, "gpu_launches": state["launches"],
        "step_us": {"losa_step_median": float(np.median(sparse_ms)) * 1e3 if sparse_ms else None,
                    "dense_first_step_median": float(np.median(dense_ms)) * 1e3 if dense_ms else None},
    }

    # ---- dominant kernel (stage-4 main kernel): eager launches of the same schedule from the next
    # block boundary, events recorded by the library immediately around that kernel
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = float(peaks.get("hbm_gbs", 6650.0))
    block0 = warm_blocks + blocks_region
    k_bytes, k_ms, kinds, k_slices = [], [], [], []
    for r in runs:
        r.layer.step.zero_()                                           # a new block starts for every layer
        r.layer.ctx.profile_stage4(True)
    for j, (b, t, n) in enumerate(sweeps):
        for r in runs[:n]:
            r.load(block0 + b, t)
            flush(j)
            r.layer.run_step_fused(r.q_s, r.k_s, r.v_s, r.m_s)
            k_ms.append(r.layer.ctx.stage4_last_ms())
            k_bytes.append(stage4_bytes(cfg, to_host(r.layer.union_pages), to_host(r.layer.union_count),
                                        to_host(r.layer.n_active), to_host(r.layer.kv_len), fp8))
            kinds.append("dense" if t == 0 else "losa")
            k_slices.append(pages_read(to_host(r.layer.union_count)))
            if t == T - 1:
                r.layer.finalize_block(r.k_s, r.v_s)
    for r in runs:
        r.layer.ctx.profile_stage4(False)
    slice_bytes = 2 * cfg.page_size * cfg.head_dim * 2
    scalable = cfg.head_dim == 128 and cfg.dtype == "bf16" and not fp8     # no ncu capture of the FP8 variant is on file

    def roof(sel):
        b = sum(x for x, k in zip(k_bytes, kinds) if k in sel)
        t = sum(x for x, k in zip(k_ms, kinds) if k in sel)
        n = sum(1 for k in kinds if k in sel)
        if not n or t <= 0:
            return None
        ach = b / (t * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "frac_of_8TBps_nominal": ach / 8000.0, "launches": n, "bytes_per_launch": b / n,
                "us_per_launch": t / n * 1e3,
                "traffic": (sum(NCU_BYTES_PER_SLICE[k] * (slice_bytes / 16384.0) * sl + NCU_FIXED_BYTES[k]
                                for k, sl in zip(kinds, k_slices) if k in sel) / n) if scalable else None,
                "peak_source": "measured (MEASURED_PEAKS.json hbm_gbs)" if peaks else "fallback 6650 GB/s"}
    result["roofline"] = roof(("losa",)) or {}
    result["roofline"]["kernel"] = ("stage-4 main kernel (paged sparse prefix attention) on the LoSA steps of the schedule: "
                                    "the graded kernel on the graded step")
    result["roofline_losa_steps"] = roof(("losa",))
    result["roofline_dense_first_step"] = roof(("dense",))
    result["roofline_all_launches"] = roof(("losa", "dense"))

    # ---- end to end through the host-buffer entry point (eager, pinned host inputs, output read back):
    # the same schedule from the next block boundary
    k = cfg.topk
    N, Bk, Hq, Hkv, d = cfg.batch, cfg.block_size, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    td = B.torch_dtype(runs[0].layer.dtype)
    pin = lambda shape: torch.empty(shape, dtype=td).pin_memory()
    es = 2 if cfg.dtype == "bf16" else 4

    def host_steps(block0):
        steps = []
        for b, t, n in sweeps:
            for l in range(n):
                inp = runs[l].block_inputs(block0 + b)[t]
                steps.append((l, t, pin((N, Bk, Hq, d)).copy_(inp.q), pin((N, Bk, Hkv, d)).copy_(inp.k_blk),
                              pin((N, Bk, Hkv, d)).copy_(inp.v_blk), inp.m_per_seq.clone()))
        return steps

    def e2e_pass(block0, n_str):
        """Every layer-step of the schedule through losa_denoise_step_host: its q / k_blk / v_blk come
        from pinned host memory and its output goes back to pinned host memory.  n_str == 1: all
        steps on one stream, strictly in order.  n_str > 1: consecutive layer-steps (different
        layers, independent here) rotate over n_str streams, a layer's steps staying on one stream.
        Host wall clock from the first call to the arrival of the last output."""
        for r in runs:
            r.layer.step.zero_()
        steps = host_steps(block0)
        streams = [torch.cuda.Stream() for _ in range(n_str)]
        stage = [tuple(torch.empty_like(x) for x in (runs[0].q_s, runs[0].k_s, runs[0].v_s)) for _ in streams]
        h_out = [pin((N, Bk, Hq, d)) for _ in streams]
        flush(0, force=True)
        torch.cuda.synchronize()
        D.barrier()
        t0 = time.perf_counter()
        for l, t, hq, hk, hv, m in steps:
            lay, j = runs[l].layer, l % n_str
            dq, dk, dv = stage[j]
            buf = B.StepBuffersT(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), lay.out.data_ptr(),
                                 lay.active_idx.data_ptr(), lay.n_active.data_ptr(), lay.topk_pages.data_ptr(),
                                 lay.union_pages.data_ptr(), lay.union_count.data_ptr())
            with torch.cuda.stream(streams[j]):
                B.losa_denoise_step_host(lay.ctx, hq, hk, hv, h_out[j], lay.kv, lay.state, buf, m, k)
                if t == T - 1:
                    lay.finalize_block(dk, dv)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        for r in runs:
            assert r.layer.ctx.poll_status() == 0
        return D.max_over_ranks(dt * 1e3, dev) / len(steps) * 1e3

    e2e_serial = e2e_pass(warm_blocks + 2 * blocks_region, 1)
    result["e2e"] = {"value": e2e_serial, "unit": UNIT, "steps": K,
                     "h2d_bytes_per_step": N * Bk * (Hq + 2 * Hkv) * d * es,
                     "d2h_bytes_per_step": N * Bk * Hq * d * es,
                     "how": "losa_denoise_step_host on pinned host q/k_blk/v_blk -> pinned host out, eager launches, every "
                            "layer-step of the schedule on one stream strictly in order (copy in, stages 1-6, copy out); host "
                            "wall clock from the first call to the arrival of the last output"
                            + (", L2 not flushed between the steps of the one layer" if L == 1 else "")}
    if L > 1:
        n_str = next(n for n in (4, 3, 2, 1) if L % n == 0)
        if n_str > 1:
            result["e2e_overlapped"] = {
                "value": e2e_pass(warm_blocks + 3 * blocks_region, n_str), "unit": UNIT, "streams": n_str,
                "how": "the same calls with consecutive layer-steps (different layers, independent in this benchmark) rotating "
                       "over several streams, so that copies and the latency-bound stages of one step overlap the kernels of "
                       "another; a throughput over independent layer-steps, not the latency of a model whose layers depend on "
                       "one another"}

    losa_pages = [p for t, p in pages if t != 0]
    result["pages_read_per_step"] = {"losa": float(np.mean(losa_pages)) if losa_pages else None,
                                     "note": "sum over sequences and KV heads of the (page, KV head) slices listed, per layer-step"}
    if rank == 0 and not args.no_extras and not fp8:
        extras(args, cfg, runs[0], lambda v: flush(v, force=True), result, warm_blocks + 4 * blocks_region)
    missing = [k2 for k2, v in (("roofline_losa_steps", result["roofline_losa_steps"]),
                                ("step_us.losa_step_median", result["step_us"]["losa_step_median"]),
                                ("pages_read_per_step.losa", result["pages_read_per_step"]["losa"])) if v is None]
    if rank == 0:
        print(json.dumps(result))
    D.shutdown()
    if missing:
        sys.exit("bench.py: no LoSA-step measurement for " + ", ".join(missing))


def extras(args, cfg, run, flush, result, block0):
    """Layer 0 only: stage breakdown, the two comparison policies on the same inputs, pages read,
    oracle timing.  Uses the two blocks after `block0`; no block is finalised here."""
    import torch
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_host
    layer, T = run.layer, cfg.steps
    q_s, k_s, v_s, m_s = run.q_s, run.k_s, run.v_s, run.m_s
    c = layer.ctx
    seq = [(block0 + j // T, j % T) for j in range(2 * T)]

    names = ["select_active", "page_scores_topk", "page_union", "sparse_prefix_attn", "block_attn_merge",
             "update_prefix_cache"]
    acc = {n: [] for n in names}
    for i, (b, t) in enumerate(seq):
        run.load(b, t)
        if t == 0:
            layer.step.zero_()
        st = layer.stage_step_arg()
        calls = [
            lambda: B.losa_select_active(c, q_s, layer.q_prev, q_s.numel() // (cfg.batch * cfg.block_size), m_s, st,
                                         layer.active_idx, layer.n_active, layer.delta),
            lambda: B.losa_page_scores_topk(c, q_s, layer.kv, layer.active_idx, layer.n_active, st, cfg.topk,
                                            layer.topk_pages, None),
            lambda: B.losa_page_union(c, layer.topk_pages, layer.active_idx, layer.n_active, cfg.topk, layer.kv_len,
                                      st, layer.union_pages, layer.union_count),
            lambda: B.losa_sparse_prefix_attn(c, q_s, layer.kv, layer.active_idx, layer.n_active, layer.union_pages,
                                              layer.union_count, layer.state),
            lambda: B.losa_block_attn_merge(c, q_s, k_s, v_s, layer.state, layer.out, layer.lse_out),
            lambda: B.losa_update_prefix_cache(c, layer.kv, layer.state, q_s, k_s, v_s, False),
        ]
        flush(i)
        for n, f in zip(names, calls):
            torch.cuda.synchronize()
            a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); f(); b2.record(); b2.synchronize()
            if t:
                acc[n].append(a.elapsed_time(b2) * 1e3)
    result["stage_us_losa_step_eager_calls"] = {n: float(np.median(v)) for n, v in acc.items() if v}

    dense_pages = int(sum((int(L) + cfg.page_size - 1) // cfg.page_size for L in to_host(layer.kv_len)) * cfg.n_kv_heads)
    result["pages_read_per_step"]["dense"] = dense_pages

    result["baselines_us_per_step_eager"] = {}
    for mode in ("naive", "dense", "losa"):
        other = layer if mode == "losa" else LosaLayer(cfg, None, None, None, layer.kv_len, mode, q_s.device, share_pool_with=layer)
        ms, pg = [], []
        for i, (b, t) in enumerate(seq):
            run.load(b, t)
            if t == 0:
                other.step.zero_()
            flush(i)
            torch.cuda.synchronize()
            a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); other.run_step(q_s, k_s, v_s, m_s); b2.record(); b2.synchronize()
            if t:
                ms.append(a.elapsed_time(b2) * 1e3)
                pg.append(pages_read(to_host(other.union_count)))
        result["baselines_us_per_step_eager"][mode] = float(np.median(ms)) if ms else None
        if mode != "losa":
            result["pages_read_per_step"][mode if mode == "naive" else "dense_measured"] = float(np.mean(pg)) if pg else None
            other.ctx.close()

    # read-only HBM probe: context for the copy-measured peak the roofline is quoted against
    probe = torch.ones(1 << 29, dtype=torch.float32, device=q_s.device)          # 2 GiB
    ts = []
    for _ in range(6):
        a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); probe.sum(); b2.record(); b2.synchronize()
        ts.append(a.elapsed_time(b2))
    result["hbm_read_probe"] = {"gbs": probe.numel() * 4 / (min(ts[1:]) * 1e-3) / 1e9,
                                "how": "torch.sum over a 2 GiB fp32 buffer, best of 5 after one warm-up"}
    del probe

    # fingerprints of layer 0's generated tensors, so that two runs can be told to have seen the same bytes
    import hashlib

    def sha(t):
        t = t.contiguous()
        if t.dtype == torch.bfloat16:
            t = t.view(torch.int16)
        return hashlib.sha256(t.cpu().numpy().tobytes()).hexdigest()
    first = run.block_inputs(block0)[0]
    result["input_sha256"] = {
        "note": f"layer 0 of this rank, after the run (blocks appended so far included); step inputs of block {block0}, step 0",
        "k_pages": sha(layer.k_pages), "v_pages": sha(layer.v_pages), "page_table": sha(layer.page_table),
        "kv_len": sha(layer.kv_len), "q": sha(first.q), "k_blk": sha(first.k_blk), "v_blk": sha(first.v_blk)}

    # the oracle on this machine's host cores (a reported baseline, not a target)
    try:
        from oracle import oracle as orc
        orc.build()
        host_w = run.w.host_copy()
        host_w.kv_len = to_host(layer.kv_len).astype(np.int32)
        host_steps = [x.host_copy() for x in run.block_inputs(block0)]
        per_step, t_dense, t_sparse, cores = oracle_block_time(cfg, host_w, host_steps)
        result["cpu_baseline"] = {
            "value": per_step * 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": (f"layer 0: one full LoSA layer-step ({t_sparse:.2f} s) and a dense first step whose prefix attention ran "
                       f"on 2 of {cfg.block_size} block tokens and was scaled x{cfg.block_size // 2} ({t_dense:.2f} s), "
                       f"averaged over a block of {T} steps")}
    except Exception as ex:  # pragma: no cover
        result["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                  "sample": f"failed: {ex}"}


def main():
    args = parse_args()
    cfg = make_config(args)
    layers = args.layers if args.layers else (36 if cfg.name == "c5" else 1)
    per_block = cfg.steps * layers
    if args.steps <= 0:
        args.steps = 4 * per_block if args.impl == "ours" else 3
    if args.warmup <= 0:
        args.warmup = per_block if args.impl == "ours" else 3
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
