#!/usr/bin/env python
"""Benchmark of the LoSA denoise-step attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c3]

One "step" is one layer-step: stages 1-6 of include/losa.h for one attention layer and one
denoising step, issued through the whole-step entry point losa_denoise_step.  Steps cycle through whole denoising blocks of the workload (step 0 of a block is
the dense first step, the others are LoSA steps).  Prints ONE JSON line.

Timing: the layer-step is captured once in a CUDA graph and replayed; each step is bracketed by
CUDA events on the launching stream; between steps, outside the timed region, the L2 is flushed by
writing a 256 MiB buffer and then reading a second one (the read pass makes the cache write its
dirty lines back, so that write-back traffic of the flush itself does not land in the timed step).  The time of K steps is the sum of the K event intervals; with several
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--active-frac", type=float, default=None, help="override the active fraction")
    ap.add_argument("--no-extras", action="store_true", help="skip baselines, stage breakdown, cpu baseline")
    return ap.parse_args()


def make_config(args):
    cfg = wl.config(args.workload)
    if args.workload == "c5":
        cfg = wl.config("c5", n_blocks=1)     # one layer of the loop; blocks restart on the same prefix
    if args.active_frac is not None:
        cfg = wl.config(args.workload, m_active=wl.active_count(args.active_frac, cfg.block_size),
                        n_blocks=cfg.n_blocks, beta_active=False)
    return cfg


def workload_name(cfg):
    lens = "/".join(f"{L // 1024}K" for L in cfg.kv_lens)
    return (f"{cfg.name}: batch {cfg.batch}, prefix {lens} tokens, pages of {cfg.page_size}, "
            f"{cfg.n_q_heads}/{cfg.n_kv_heads} heads x {cfg.head_dim}, block {cfg.block_size}, "
            f"{cfg.steps} steps/block, {cfg.m_active} active tokens/step, top-{cfg.topk} pages, {cfg.dtype}")


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
def stage4_bytes(cfg, up, uc, na, kv_len):
    """Algorithmic bytes of one stage-4 launch: K and V of the valid tokens of every listed page,
    the active queries, the union list and page-table entries read, the state rows written."""
    e = 2 if cfg.dtype == "bf16" else 4
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
            total += 2 * toks * d * e + 8 * n
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
        "config": {"workload": workload_name(cfg)},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg):
    import torch
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200 import build as build_mod
    from paper_2604_12056_b200 import dist as D
    from paper_2604_12056_b200.layer import LosaLayer, to_device, to_host

    local = D.env_rank()[2]
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rank, world, local = D.init("nccl", dev)
    if not os.path.exists(B.LIB_PATH):
        if local == 0:
            build_mod.build()
        D.barrier()

    w = wl.Workload(cfg, replica=D.replica_of(rank))
    layer = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, "losa", dev)
    T = cfg.steps
    total = args.warmup + args.steps
    n_blocks = (total + T - 1) // T
    host_steps = []
    for _ in range(n_blocks):
        host_steps += w.block_steps()
    host_steps = host_steps[:total]
    dev_steps = [(to_device(i.q, dev), to_device(i.k_blk, dev), to_device(i.v_blk, dev), to_device(i.m_per_seq, dev))
                 for i in host_steps]
    q_s, k_s, v_s = (torch.empty_like(t) for t in dev_steps[0][:3])
    m_s = torch.empty_like(dev_steps[0][3])
    flush_w = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)   # fp32: sum() reads it in place

    class _Flush:
        """Evicts the L2 (write > L2, then read > L2 so that no dirty lines are left behind)."""
        def fill_(self, v):
            flush_w.fill_(v)
            flush_r.sum()
    flush = _Flush()

    def load(i):
        q, k, v, m = dev_steps[i]
        q_s.copy_(q); k_s.copy_(k); v_s.copy_(v); m_s.copy_(m)
        if i % T == 0:
            layer.step.zero_()          # a new block starts: no valid cache

    # eager warm-up of every kernel (tensor maps, attributes, second stream), then capture the
    # whole-step call
    load(0)
    layer.run_step_fused(q_s, k_s, v_s, m_s)
    torch.cuda.synchronize()
    assert layer.ctx.poll_status() == 0
    n0 = layer.ctx.launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        layer.run_step_fused(q_s, k_s, v_s, m_s)
    launches_per_step = layer.ctx.launch_count() - n0

    def timed_pass(first, count, record_pages=None):
        evs = []
        for i in range(first, first + count):
            load(i)
            flush.fill_(i & 0xff)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            evs.append((a, b))
            if record_pages is not None:
                record_pages.append((i % T, pages_read(to_host(layer.union_count))))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    timed_pass(0, args.warmup)
    D.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    pages = []
    ms = timed_pass(args.warmup, args.steps, pages)
    torch.cuda.synchronize()
    D.barrier()
    clocks = sampler.stop()
    assert layer.ctx.poll_status() == 0
    total_ms = D.max_over_ranks(float(sum(ms)), dev)
    ms_per_step = total_ms / args.steps
    sparse_ms = [x for x, (t, _) in zip(ms, pages) if t != 0]
    dense_ms = [x for x, (t, _) in zip(ms, pages) if t == 0]

    result = {
        "metric": METRIC, "value": ms_per_step * 1e3, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sequences_per_gpu": cfg.batch,
                   "launch": "CUDA graph replay of losa_denoise_step (stages 1-6 in one call)",
                   "l2": "flushed between steps, outside the timed region: 256 MiB write, then 256 MiB read so no dirty lines remain"},
        "clocks": clocks, "gpu_launches": launches_per_step * args.steps,
        "step_us": {"losa_step_median": float(np.median(sparse_ms)) * 1e3 if sparse_ms else None,
                    "dense_first_step_median": float(np.median(dense_ms)) * 1e3 if dense_ms else None},
    }

    # ---- dominant kernel (stage-4 main kernel), eager launches of the same steps, events around it
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = float(peaks.get("hbm_gbs", 6650.0))
    layer.ctx.profile_stage4(True)
    k_bytes, k_ms, kinds = [], [], []
    first = args.warmup - (args.warmup % T)       # start at a block boundary
    first = first if first + args.steps <= total else 0
    for i in range(first, min(total, first + max(args.steps, T))):
        load(i)
        flush.fill_(i & 0xff)
        layer.run_step_fused(q_s, k_s, v_s, m_s)
        k_ms.append(layer.ctx.stage4_last_ms())
        k_bytes.append(stage4_bytes(cfg, to_host(layer.union_pages), to_host(layer.union_count),
                                    to_host(layer.n_active), to_host(layer.kv_len)))
        kinds.append("dense" if i % T == 0 else "losa")
    layer.ctx.profile_stage4(False)

    # DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of this kernel, from the
    # ncu capture summarised in profiles/attn_mma_kernel_c3.txt (same command, workload c3 only)
    ncu_traffic = {"losa": 162.49e6 + 5.42e6, "dense": 438.54e6 + 6.88e6} if cfg.name == "c3" and args.active_frac is None else None

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
                "traffic": (sum(ncu_traffic[k] for k in kinds if k in sel) / n) if ncu_traffic else None,
                "peak_source": "measured (MEASURED_PEAKS.json hbm_gbs)" if peaks else "fallback 6650 GB/s"}
    result["roofline"] = roof(("losa", "dense")) or {}
    result["roofline"]["kernel"] = "stage-4 main kernel (paged prefix attention), every launch of whole blocks"
    result["roofline_losa_steps"] = roof(("losa",))
    result["roofline_dense_first_step"] = roof(("dense",))

    # ---- end to end through the host-buffer entry point
    k = cfg.topk
    N, Bk, Hq, Hkv, d = cfg.batch, cfg.block_size, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    td = B.torch_dtype(layer.dtype)
    pin = lambda shape: torch.empty(shape, dtype=td).pin_memory()
    h_q, h_k, h_v, h_o = pin((N, Bk, Hq, d)), pin((N, Bk, Hkv, d)), pin((N, Bk, Hkv, d)), pin((N, Bk, Hq, d))
    d_q, d_k, d_v = torch.empty_like(q_s), torch.empty_like(k_s), torch.empty_like(v_s)
    buf = B.StepBuffersT(d_q.data_ptr(), d_k.data_ptr(), d_v.data_ptr(), layer.out.data_ptr(),
                         layer.active_idx.data_ptr(), layer.n_active.data_ptr(), layer.topk_pages.data_ptr(),
                         layer.union_pages.data_ptr(), layer.union_count.data_ptr())
    e2e_ms = []
    host_t = []
    for i in range(total):
        q, kk, vv, m = dev_steps[i]
        h_q.copy_(q.cpu()); h_k.copy_(kk.cpu()); h_v.copy_(vv.cpu()); m_s.copy_(m)
        if i % T == 0:
            layer.step.zero_()
        flush.fill_(i & 0xff)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        a.record()
        B.losa_denoise_step_host(layer.ctx, h_q, h_k, h_v, h_o, layer.kv, layer.state, buf, m_s, k)
        b.record()
        b.synchronize()
        host_t.append(time.perf_counter() - t0)
        if i >= args.warmup:
            e2e_ms.append(max(a.elapsed_time(b), 0.0))
    assert layer.ctx.poll_status() == 0
    e2e_total = D.max_over_ranks(float(sum(host_t[args.warmup:])) * 1e3, dev)   # host wall clock of the K calls incl. sync
    es = 2 if cfg.dtype == "bf16" else 4
    result["e2e"] = {"value": e2e_total / args.steps * 1e3, "unit": UNIT,
                     "h2d_bytes_per_step": N * Bk * (Hq + 2 * Hkv) * d * es,
                     "d2h_bytes_per_step": N * Bk * Hq * d * es,
                     "device_span_us": float(np.mean(e2e_ms)) * 1e3,
                     "how": "losa_denoise_step_host on pinned host q/k_blk/v_blk -> host out, eager launches, "
                            "host wall clock per call including the final synchronise"}

    if rank == 0 and not args.no_extras:
        extras(args, cfg, w, layer, host_steps, dev_steps, load, flush, (q_s, k_s, v_s, m_s), result, pages)
    if rank == 0:
        print(json.dumps(result))
    D.shutdown()


def extras(args, cfg, w, layer, host_steps, dev_steps, load, flush, static, result, pages):
    """Stage breakdown, the two comparison policies on the same inputs, pages read, oracle timing."""
    import torch
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_host
    q_s, k_s, v_s, m_s = static
    T = cfg.steps
    c = layer.ctx

    # per-stage device time of LoSA steps (eager, one synchronise before each call)
    names = ["select_active", "page_scores_topk", "page_union", "sparse_prefix_attn", "block_attn_merge",
             "update_prefix_cache"]
    acc = {n: [] for n in names}
    for i in range(min(len(dev_steps), 2 * T)):
        load(i)
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
        flush.fill_(i & 0xff)
        for n, f in zip(names, calls):
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); f(); b.record(); b.synchronize()
            if i % T:
                acc[n].append(a.elapsed_time(b) * 1e3)
    result["stage_us_losa_step"] = {n: float(np.median(v)) for n, v in acc.items() if v}

    # pages read per step (sum over sequences and KV heads of the union size)
    dense_pages = int(sum((int(L) + cfg.page_size - 1) // cfg.page_size for L in cfg.kv_lens) * cfg.n_kv_heads)
    losa_pages = [p for t, p in pages if t != 0]
    result["pages_read_per_step"] = {"losa": float(np.mean(losa_pages)) if losa_pages else None, "dense": dense_pages}

    # naive per-query sparse attention and dense prefix attention, same inputs, same calls
    for mode in ("naive", "dense"):
        other = LosaLayer(cfg, None, None, None, layer.kv_len, mode, q_s.device, share_pool_with=layer)
        ms, pg = [], []
        for i in range(min(len(dev_steps), 2 * T)):
            q, k, v, m = dev_steps[i]
            q_s.copy_(q); k_s.copy_(k); v_s.copy_(v); m_s.copy_(m)
            if i % T == 0:
                other.step.zero_()
            flush.fill_(i & 0xff)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); other.run_step(q_s, k_s, v_s, m_s); b.record(); b.synchronize()
            if i % T:
                ms.append(a.elapsed_time(b) * 1e3)
                pg.append(pages_read(to_host(other.union_count)))
        result.setdefault("baselines_us_per_step_eager", {})[mode] = float(np.median(ms)) if ms else None
        result["pages_read_per_step"][mode if mode == "naive" else "dense_measured"] = float(np.mean(pg)) if pg else None
        other.ctx.close()
    # LoSA eager for a like-for-like comparison with the two eager baselines above
    ms = []
    for i in range(min(len(dev_steps), 2 * T)):
        load(i)
        flush.fill_(i & 0xff)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); layer.run_step(q_s, k_s, v_s, m_s); b.record(); b.synchronize()
        if i % T:
            ms.append(a.elapsed_time(b) * 1e3)
    result["baselines_us_per_step_eager"]["losa"] = float(np.median(ms)) if ms else None

    # the oracle on this machine's host cores (a reported baseline, not a target)
    try:
        from oracle import oracle as orc
        orc.build()
        per_step, t_dense, t_sparse, cores = oracle_block_time(cfg, w, host_steps[:T])
        result["cpu_baseline"] = {
            "value": per_step * 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": (f"one full LoSA layer-step ({t_sparse:.2f} s) and a dense first step whose prefix attention ran "
                       f"on 2 of {cfg.block_size} block tokens and was scaled x{cfg.block_size // 2} ({t_dense:.2f} s), "
                       f"averaged over a block of {T} steps")}
    except Exception as ex:  # pragma: no cover
        result["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                  "sample": f"failed: {ex}"}


def main():
    args = parse_args()
    if args.warmup < 3:
        args.warmup = 3
    cfg = make_config(args)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
