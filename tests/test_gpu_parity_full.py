"""GPU-vs-oracle parity at the full sizes of the benchmark configurations (needs a B200).

A LoSA step recomputes only the active tokens, so the oracle follows it in full at any prefix
length; a dense first step is compared in full where the oracle finishes in seconds (8K prefix)
and on sampled block tokens otherwise.  Index outputs are always compared in full and exactly.
"""
import numpy as np
import pytest

from helpers import OracleLayer
from paper_2604_12056_b200 import workloads as wl
from test_gpu_parity import assert_close, assert_lse_close, compare, run_blocks

pytestmark = pytest.mark.gpu


def dense_step_on_samples(g, o, inp, sample, what):
    """Step 0 of a block on the GPU (six calls or the whole-step call); the oracle recomputes the
    prefix statistics of the sampled block tokens one by one and takes the GPU's values for the
    others (they are within tolerance or the sampled comparison would have failed), so that the
    following steps can be compared in full."""
    from oracle import oracle as orc
    cfg, sh = g.cfg, o.sh
    N, B = cfg.batch, cfg.block_size
    s0 = g.snapshot()
    assert g.ctx.poll_status() == 0
    act, na, _ = orc.select_active(sh, inp.q, o.q_prev, inp.m_per_seq, o.step)
    up, uc = orc.page_union(sh, o.topk, act, na, cfg.topk, o.kv_len, o.step)
    for key, ref in (("act", act), ("na", na), ("up", up), ("uc", uc)):
        assert (s0[key] == ref).all(), f"{what}: {key}"
    sample = np.asarray(sample, np.int32)
    act_s = np.full((N, B), -1, np.int32)
    act_s[:, :sample.size] = sample
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    orc.sparse_prefix_attn(sh, inp.q, o.kv, act_s, np.full(N, sample.size, np.int32), up, uc, o.o_p, o.lse_p)
    assert_close(s0["o_p"][:, sample], o.o_p[:, sample], cfg.dtype, what + " sampled o_p")
    assert_lse_close(s0["lse_p"][:, sample], o.lse_p[:, sample], what + " sampled lse_p")
    out, lse = orc.block_attn_merge(sh, inp.q, inp.k_blk, inp.v_blk, o.o_p, o.lse_p)
    assert_close(s0["out"], out, cfg.dtype, what + " out")
    assert_lse_close(s0["lse"], lse, what + " lse")
    orc.update_prefix_cache(sh, o.kv, o.q_prev, o.step, inp.q, inp.k_blk, inp.v_blk, False)
    return uc


@pytest.mark.parametrize("fused", [False, True])
def test_full_size_c2_whole_block(fused):
    """8,192-token prefix, 256 pages of 32, top-32 pages, three active tokens: every step of a
    block in full, the dense first step included; the comparison policies on the six-call path."""
    run_blocks(wl.config("c2"), modes=("losa",) if fused else ("losa", "naive", "dense"), fused=fused,
               want_scores=not fused)


@pytest.mark.parametrize("fused", [False, True])
def test_full_size_c4_very_long_context(fused):
    """131,072-token prefix in 2,048 pages of 64, block of 64 tokens (two row groups per KV head),
    five active tokens, top-64 pages, 5 % heavy-hitter pages: the dense first step on sampled tokens
    of both row groups, then three LoSA steps in full.  2,048 pages per list: the top-k selection
    re-reads its score rows (they do not fit the registers of one CTA)."""
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c4", steps=4)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    o = OracleLayer(w)
    steps = w.block_steps()
    dev = lambda i: (to_device(i.q), to_device(i.k_blk), to_device(i.v_blk), to_device(i.m_per_seq))
    run = g.run_step_fused if fused else g.run_step
    run(*dev(steps[0]))
    dense_step_on_samples(g, o, steps[0], [5, 40, 63], "c4 dense step")
    dense_pages = cfg.n_kv_heads * 2048
    for t in range(1, cfg.steps):
        run(*dev(steps[t]))
        snap = g.snapshot()
        assert g.ctx.poll_status() == 0
        ref = o.run_step(steps[t])
        if fused:
            snap["delta"] = ref["delta"]
        assert ref["act"][0, :cfg.m_active].tolist() == steps[t].planted[0].tolist()
        compare(snap, ref, cfg, f"c4 full size, LoSA step {t}")
        assert cfg.n_kv_heads * 64 <= ref["uc"].sum() < dense_pages // 4


def test_full_size_c5_second_block_after_append():
    """The benchmark's default workload from its second block on: 32,800-token prefixes, i.e. 1,025
    pages of 32 per sequence (more than the 1,024 scores a top-k CTA keeps in registers), per-head
    lists.  One layer generated on the
    device as the benchmark does; block 0 runs its dense step and one LoSA step and is finalised
    (appended); block 1's dense step is compared on samples, its LoSA step in full."""
    import torch
    from paper_2604_12056_b200.layer import LosaLayer
    cfg = wl.config("c5", n_blocks=2)
    dw = wl.DeviceWorkload(cfg, replica=0, layer=3)
    g = LosaLayer(cfg, dw.k_pages, dw.v_pages, dw.page_table, dw.kv_len)
    a0, a1 = dw.start_block(), dw.next_step()
    for a in (a0, a1):
        g.run_step_fused(a.q, a.k_blk, a.v_blk, a.m_per_seq)
    g.finalize_block(a1.k_blk, a1.v_blk)
    torch.cuda.synchronize()
    assert g.ctx.poll_status() == 0
    g.topk_pages.fill_(-9)       # rows of stable tokens are never written: same start as the fresh oracle layer below
    # the oracle starts from the grown cache: a host copy of the pool after the append, its own summaries
    host = dw.host_copy()
    host.kv_len = g.snapshot()["kv_len"].astype(np.int32)
    assert (host.kv_len == 32768 + 32).all()
    o = OracleLayer(host)
    from paper_2604_12056_b200.layer import to_host
    used = to_host(g.page_table)[:, :1025].reshape(-1)
    assert (to_host(g.kmin)[used] == wl.elem_to_f32(o.kmin)[used]).all()
    assert (to_host(g.kmax)[used] == wl.elem_to_f32(o.kmax)[used]).all()
    b0, b1 = dw.start_block(), dw.next_step()
    g.run_step_fused(b0.q, b0.k_blk, b0.v_blk, b0.m_per_seq)
    torch.cuda.synchronize()
    uc = dense_step_on_samples(g, o, b0.host_copy(), [7, 30], "c5 block 1 dense step")
    assert (uc == 1025).all()
    g.run_step_fused(b1.q, b1.k_blk, b1.v_blk, b1.m_per_seq)
    torch.cuda.synchronize()
    snap = g.snapshot()
    assert g.ctx.poll_status() == 0
    h1 = b1.host_copy()
    ref = o.run_step(h1)
    snap["delta"] = ref["delta"]
    compare(snap, ref, cfg, "c5 block 1 (1,025 pages), LoSA step")
    # the appended page is a candidate like any other: it must be scored (its id may or may not be chosen)
    assert ref["topk"][ref["topk"] >= 0].max() <= 1024
