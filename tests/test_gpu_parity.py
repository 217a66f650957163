"""GPU-vs-oracle parity of every stage, through the C-ABI (needs a B200).

Index outputs (active sets, top-k page lists, unions, counters) must be bit-exact; attention
outputs within the stated tolerances: fp32 mode |a-b| <= 1e-5 * max(|b|, max|b_row|); bf16 mode
|a-b| <= 2e-2 + 1e-2 |b|; every LSE within 1e-3.
"""
import numpy as np
import pytest

from helpers import OracleLayer, delta_gap_ok, tau_gap_ok
from paper_2604_12056_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def assert_close(got, want, dtype, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    if dtype == "f32":
        row_max = np.abs(want).max(axis=-1, keepdims=True)
        tol = 1e-5 * np.maximum(np.abs(want), row_max)
    else:
        tol = 2e-2 + 1e-2 * np.abs(want)
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, worst {np.abs(got - want).max():.3e}"


def assert_lse_close(got, want, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    inf = np.isinf(want)
    assert (np.isinf(got) == inf).all() and (got[inf] == want[inf]).all(), what
    assert (np.abs(got[~inf] - want[~inf]) <= 1e-3).all(), f"{what}: worst {np.abs(got[~inf] - want[~inf]).max():.3e}"


def compare(snap, ref, cfg, what, tau=0.0):
    for key in ("act", "na", "topk", "up", "uc"):
        assert (snap[key] == ref[key]).all(), f"{what}: {key} differs"
    np.testing.assert_allclose(snap["delta"], ref["delta"], rtol=1e-5, atol=1e-12, err_msg=what)
    for s in range(cfg.batch):
        m = int(ref["na"][s])
        if tau > 0.0 and m < cfg.block_size:
            assert tau_gap_ok(ref["delta"][s], m, tau), f"{what}: threshold-ambiguous Delta in sequence {s}"
        else:
            assert delta_gap_ok(ref["delta"][s], m), f"{what}: selection-ambiguous Delta in sequence {s}"
    assert_close(snap["o_p"], ref["o_p"], cfg.dtype, what + " o_p")
    assert_lse_close(snap["lse_p"], ref["lse_p"], what + " lse_p")
    assert_close(snap["out"], ref["out"], cfg.dtype, what + " out")
    assert_lse_close(snap["lse"], ref["lse"], what + " lse")


def run_blocks(cfg, modes=("losa",), m=None, n_blocks=1, pad_nan=True, want_scores=True, fused=False, tau=0.0,
               pooled=False, state_bf16=False):
    """Runs n_blocks blocks through GPU and oracle in lock-step, comparing after every step."""
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    w = wl.Workload(cfg, pad_nan=pad_nan)
    gpu = {md: LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, md, tau=tau, pooled=pooled,
                         state_bf16=state_bf16) for md in modes}
    ora = {md: OracleLayer(w, md, tau=tau, pooled=pooled, state_bf16=state_bf16) for md in modes}
    for md in modes:     # page summaries: exact min / max on both sides
        from paper_2604_12056_b200.layer import to_host
        P = [(int(L) + cfg.page_size - 1) // cfg.page_size for L in w.kv_len]
        used = np.concatenate([w.page_table[s, :P[s]] for s in range(cfg.batch)]) if sum(P) else np.zeros(0, np.int64)
        assert (to_host(gpu[md].kmin)[used] == wl.elem_to_f32(ora[md].kmin)[used]).all()
        assert (to_host(gpu[md].kmax)[used] == wl.elem_to_f32(ora[md].kmax)[used]).all()
    for b in range(n_blocks):
        steps = w.block_steps(m)
        for t, inp in enumerate(steps):
            last = t == len(steps) - 1 and n_blocks > 1
            q, kb, vb = to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk)
            mt = to_device(inp.m_per_seq)
            for md in modes:
                g = gpu[md]
                if fused:
                    g.run_step_fused(q, kb, vb, mt)
                else:
                    g.run_step(q, kb, vb, mt, want_scores=want_scores)
                snap = g.snapshot()

                assert g.ctx.poll_status() == 0
                ref = ora[md].run_step(inp, finalize=last)
                if fused:
                    snap["delta"] = ref["delta"]          # the whole-step call does not export Delta
                compare(snap, ref, cfg, f"{cfg.name}/{md} block {b} step {t}", tau if md == "losa" else 0.0)
                if want_scores and not fused and md == "losa" and t > 0:
                    sel = ref["topk"] >= 0
                    rows = np.zeros_like(sel)
                    for s in range(cfg.batch):
                        rows[s, ref["act"][s, :ref["na"][s]]] = True
                    assert np.isfinite(snap["topk_scores"][sel & rows]).all()
                if last:
                    g.finalize_block(kb, vb)
                    s2 = g.snapshot()
                    assert (s2["kv_len"] == ora[md].kv_len).all() and (s2["step"] == 0).all()
                    assert g.ctx.poll_status() == 0
    return gpu, ora


def test_c1_fp32_full_block_all_modes():
    run_blocks(wl.config("c1"), modes=("losa", "naive", "dense"))


def test_c1_hidden_state_selection():
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c1")
    w = wl.Workload(cfg)
    steps = w.block_steps()
    g, o = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len), OracleLayer(w)
    args = lambda i: (to_device(i.q), to_device(i.k_blk), to_device(i.v_blk), to_device(i.m_per_seq))
    g.run_step(*args(steps[0]))
    o.run_step(steps[0])
    g.run_step(*args(steps[1]), x_sel=(to_device(steps[1].hidden), to_device(steps[0].hidden)))
    ref = o.run_step(steps[1], x_sel=(steps[1].hidden, steps[0].hidden))
    compare(g.snapshot(), ref, cfg, "c1 hidden-state selection")
    assert ref["act"][0, :4].tolist() == steps[1].planted[0].tolist()


def test_c2_reduced_bf16_all_modes():
    run_blocks(wl.config("c2", kv_lens=(2048,), steps=4), modes=("losa", "naive", "dense"))


@pytest.mark.parametrize("g,d,hq,hkv,dtype", [
    (16, 64, 4, 1, "bf16"), (32, 128, 8, 2, "bf16"), (64, 128, 8, 8, "bf16"), (16, 128, 16, 1, "bf16"),
    (32, 64, 6, 2, "f32"), (64, 128, 4, 2, "f32"), (16, 128, 2, 2, "f32"), (32, 128, 28, 4, "bf16"),
])
def test_ragged_batch_partial_pages_and_empty_prefix(g, d, hq, hkv, dtype):
    # ragged lengths: a partial last page, an empty prefix, a single token, exact page multiples
    cfg = wl.config("c2", n_q_heads=hq, n_kv_heads=hkv, head_dim=d, page_size=g, dtype=dtype,
                    kv_lens=(5 * g + 3, 0, 1, 7 * g), block_size=12, steps=3, topk=3, m_active=2)
    run_blocks(cfg, modes=("losa", "naive"))


@pytest.mark.parametrize("g,d", [(16, 64), (16, 128), (32, 64), (64, 64)])
def test_page_groups_of_the_tensor_core_kernel(g, d):
    # the bf16 stage-4 kernel takes pages in groups of 128 tokens: several whole groups, a last group
    # with fewer pages (also one that ends inside a 32-column chunk), a partial last page with NaN
    # behind it, every page listed (dense mode) and few listed (LoSA)
    cfg = wl.config("c2", n_q_heads=8, n_kv_heads=2, head_dim=d, page_size=g, kv_lens=(21 * g + 5, 9 * g, 128 + g),
                    block_size=16, steps=3, topk=6, m_active=3)
    run_blocks(cfg, modes=("losa", "dense"))


@pytest.mark.parametrize("tau", [0.3, 0.5, 0.9])
def test_threshold_pruning_rule_whole_blocks(tau):
    # stage 1 keeps tokens until their Delta reach tau of the block's total; everything downstream
    # follows the active set it produces (bf16 and fp32, two sequences)
    run_blocks(wl.config("c2", kv_lens=(1500, 700), steps=4, block_size=16, topk=6), tau=tau)
    run_blocks(wl.config("c1", kv_lens=(300, 180), steps=3), tau=tau)


@pytest.mark.parametrize("fused", [False, True])
def test_pooled_selector_whole_blocks(fused):
    # one page list per (token, KV head): six-call path and whole-step call, bf16 with G = 4 and fp32 with G = 3
    run_blocks(wl.config("c2", kv_lens=(2048, 1500), steps=4), modes=("losa",) if fused else ("losa", "naive"),
               pooled=True, fused=fused, want_scores=not fused)
    cfg = wl.config("c2", n_q_heads=6, n_kv_heads=2, head_dim=64, page_size=16, dtype="f32",
                    kv_lens=(5 * 16 + 3, 0, 1, 7 * 16), block_size=12, steps=3, topk=3, m_active=2)
    run_blocks(cfg, pooled=True, fused=fused, want_scores=not fused)


@pytest.mark.parametrize("pooled", [True, False])
@pytest.mark.parametrize("pages,topk", [(700, 600), (1100, 8), (1300, 8), (1100, 600)])
def test_long_lists_and_large_budgets(pages, topk, pooled):
    # k > 512 pages takes the whole-list sort; more than 1024 pages the selection that re-reads its
    # row of scores or bounds instead of keeping it in registers: per-head lists and pooled lists go through both
    cfg = wl.config("c2", n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, kv_lens=(16 * pages,),
                    block_size=4, steps=2, topk=topk, m_active=2)
    run_blocks(cfg, pooled=pooled)


def test_whole_step_call_beyond_the_bitmap_of_the_selection_kernel():
    # more than 8,192 pages per sequence: the whole-step call's selection kernel leaves stage 3 to the
    # union kernel (its bitmap holds 256 words); lists, union and attention as usual
    cfg = wl.config("c2", n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, kv_lens=(16 * 8300 + 3,),
                    block_size=4, steps=2, topk=8, m_active=2)
    assert cfg.max_pages_per_seq > 8192
    run_blocks(cfg, modes=("losa",), fused=True, want_scores=False)


@pytest.mark.parametrize("kw", [
    dict(kv_lens=(2048, 1500), steps=4),
    dict(n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, kv_lens=(16 * 1100 + 5, 700), block_size=8, steps=3, topk=8,
         m_active=3),
    dict(kv_lens=(150,), block_size=8, steps=3, topk=64, m_active=2),
])
@pytest.mark.parametrize("fused", [False, True])
def test_tensor_core_selector_under_the_relaxed_list_rule(kw, fused):
    """losa_page_scores_topk_mma: page scores as a GEMM on the tensor cores.  Its lists are checked
    against the relaxed validity rule (fp64 scores, slack 2^-11 of the largest term magnitude sum);
    everything downstream is compared as usual, the oracle taking the GPU's own lists: the union
    exactly, the attention within the usual tolerances."""
    from oracle import oracle as orc
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", **kw)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, mma_selector=True)
    o = OracleLayer(w)
    sh, k = o.sh, cfg.topk
    same = total = 0
    for t, inp in enumerate(w.block_steps()):
        args = (to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk), to_device(inp.m_per_seq))
        if fused:                                  # the whole-step call with losa_set_step_selector(ctx, LOSA_SELECTOR_MMA)
            g.run_step_fused(*args)
        else:
            g.run_step(*args)
        snap = g.snapshot()
        assert g.ctx.poll_status() == 0
        act, na, _ = orc.select_active(sh, inp.q, o.q_prev, inp.m_per_seq, o.step)
        assert (snap["act"] == act).all() and (snap["na"] == na).all()
        if t > 0:
            assert orc.check_topk_relaxed(sh, inp.q, o.kv, act, na, k, snap["topk"], 2.0 ** -11, o.step) == 0
            exact = np.full_like(snap["topk"], -9)
            orc.page_scores_topk(sh, inp.q, o.kv, act, na, k, o.step, topk_pages=exact)
            for s in range(cfg.batch):
                for tok in act[s, :na[s]]:
                    total += cfg.n_q_heads
                    same += int((np.sort(exact[s, tok], -1) == np.sort(snap["topk"][s, tok], -1)).all(-1).sum())
        up, uc = orc.page_union(sh, snap["topk"], act, na, k, o.kv_len, o.step)
        assert (snap["up"] == up).all() and (snap["uc"] == uc).all()
        orc.sparse_prefix_attn(sh, inp.q, o.kv, act, na, up, uc, o.o_p, o.lse_p)
        out, lse = orc.block_attn_merge(sh, inp.q, inp.k_blk, inp.v_blk, o.o_p, o.lse_p)
        what = f"tensor-core selector, step {t}"
        assert_close(snap["o_p"], o.o_p, cfg.dtype, what + " o_p")
        assert_lse_close(snap["lse_p"], o.lse_p, what + " lse_p")
        assert_close(snap["out"], out, cfg.dtype, what + " out")
        assert_lse_close(snap["lse"], lse, what + " lse")
        orc.update_prefix_cache(sh, o.kv, o.q_prev, o.step, inp.q, inp.k_blk, inp.v_blk, False)
    assert same >= 0.9 * total          # as sets, nearly all lists are the exact ones


def test_tensor_core_selector_needs_bf16():
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c1", kv_lens=(64,), steps=2)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, mma_selector=True)
    inp = w.start_block()
    with pytest.raises(B.LosaError) as e:
        g.run_step(to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk), to_device(inp.m_per_seq))
    assert e.value.code == B.LOSA_ERR_UNSUPPORTED


@pytest.mark.parametrize("name", ["p1", "p2"])
def test_paper_shaped_workloads_reduced(name):
    # the shapes of the paper's latency study (batch 1, five active tokens, budget 16 pages), shorter prefix
    run_blocks(wl.config(name, kv_lens=(4096 + 77,), steps=4), modes=("losa", "naive", "dense"))


def test_more_segments_than_ctas_and_very_short_segments():
    # 24 sequences x 8 KV heads = 192 (sequence, KV head) segments for the 148 CTAs of the bf16
    # stage-4 kernel, most of them a page or two long (shorter than the pad the work list charges per
    # segment), some empty: CTAs whose share holds no page at all, CTAs that cross several segments
    lens = tuple(0 if i in (3, 17) else 1 + (13 * i) % 90 for i in range(24))
    cfg = wl.config("c2", n_q_heads=16, n_kv_heads=8, head_dim=64, page_size=16, kv_lens=lens,
                    block_size=8, steps=3, topk=2, m_active=2)
    run_blocks(cfg, modes=("losa", "dense"))
    run_blocks(cfg, modes=("losa",), fused=True, want_scores=False)


@pytest.mark.parametrize("fused", [False, True])
def test_sequences_without_active_tokens_beside_others(fused):
    # per-sequence active counts 0 / 3 / 1 / 0 in one batch: the stage-2 work list walks every
    # sequence that is past its first step, with or without active tokens
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", kv_lens=(40 * 32 + 5, 300, 129 * 32, 64), block_size=16, steps=4, topk=6, m_active=3)
    w = wl.Workload(cfg)
    g, o = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len), OracleLayer(w)
    for t, inp in enumerate(w.block_steps()):
        if t > 0:
            inp.m_per_seq[:] = np.array([0, 3, 1, 0], np.int32)
        args = tuple(to_device(x) for x in (inp.q, inp.k_blk, inp.v_blk, inp.m_per_seq))
        if fused:
            g.run_step_fused(*args)
        else:
            g.run_step(*args)
        snap, ref = g.snapshot(), o.run_step(inp)
        assert g.ctx.poll_status() == 0
        if fused:
            snap["delta"] = ref["delta"]
        compare(snap, ref, cfg, f"mixed active counts step {t}")
        if t > 0:
            assert ref["na"].tolist() == [0, 3, 1, 0]


@pytest.mark.parametrize("pooled", [False, True])
@pytest.mark.parametrize("fused", [False, True])
def test_sequences_on_different_steps_in_one_batch(fused, pooled):
    # the step counter is per sequence: after two steps, sequences 0 and 2 are put back on a first step
    # (every token active, union = whole prefix) while 1 and 3 go on with lists; then all continue
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", kv_lens=(40 * 32 + 5, 300, 70 * 32, 64), block_size=16, steps=5, topk=6, m_active=3)
    w = wl.Workload(cfg)
    g, o = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, pooled=pooled), OracleLayer(w, pooled=pooled)
    for t, inp in enumerate(w.block_steps()):
        if t == 2:
            g.step[0] = 0
            g.step[2] = 0
            o.step[[0, 2]] = 0
        args = tuple(to_device(x) for x in (inp.q, inp.k_blk, inp.v_blk, inp.m_per_seq))
        if fused:
            g.run_step_fused(*args)
        else:
            g.run_step(*args)
        snap, ref = g.snapshot(), o.run_step(inp)
        assert g.ctx.poll_status() == 0
        if fused:
            snap["delta"] = ref["delta"]
        compare(snap, ref, cfg, f"staggered steps, step {t}")
        if t == 2:
            assert ref["na"].tolist() == [16, 3, 16, 3]
            P = [(L + 31) // 32 for L in cfg.kv_lens]
            assert (ref["uc"][0] == P[0]).all() and (ref["uc"][2] == P[2]).all() and (ref["uc"][1] <= P[1]).all()


@pytest.mark.parametrize("fused", [False, True])
def test_state_stored_in_bf16(fused):
    # the cached prefix output stored rounded to bf16: the oracle rounds the rows stage 4 writes, and
    # the merge of the same step and the reuse in later steps see the rounded values on both sides
    cfg = wl.config("c2", kv_lens=(33 * 32 + 7, 500), block_size=16, steps=4, topk=6, m_active=3, n_blocks=2)
    gpu, _ = run_blocks(cfg, modes=("losa",) if fused else ("losa", "dense"), n_blocks=2, fused=fused, want_scores=False,
                        state_bf16=True)
    import torch
    assert gpu["losa"].o_p.dtype == torch.bfloat16


def test_bf16_state_needs_a_bf16_context():
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c1")
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, state_bf16=True)
    inp = w.start_block()
    with pytest.raises(B.LosaError) as e:
        g.run_step(*(to_device(x) for x in (inp.q, inp.k_blk, inp.v_blk, inp.m_per_seq)))
    assert e.value.code == B.LOSA_ERR_UNSUPPORTED


@pytest.mark.parametrize("m", [0, 1, 16])
def test_active_count_extremes(m):
    cfg = wl.config("c2", kv_lens=(700, 333), block_size=16, steps=3, topk=4, m_active=max(m, 1))
    run_blocks(cfg, m=m)


def test_budget_larger_than_cache_and_shuffled_pages():
    cfg = wl.config("c2", kv_lens=(150,), block_size=8, steps=3, topk=64, m_active=2)
    gpu, _ = run_blocks(cfg)
    assert gpu["losa"].snapshot()["uc"].max() == 5


def test_maximum_block_two_row_groups():
    # B = 64 tokens x 4 heads per KV head = 256 query rows: two row groups per (sequence, KV head)
    cfg = wl.config("c4", kv_lens=(64 * 40 + 17,), steps=2, topk=8, m_active=40, heavy_frac=0.0)
    run_blocks(cfg, modes=("losa", "dense"))


def test_many_rows_per_kv_head_fp32():
    cfg = wl.config("c1", n_q_heads=16, n_kv_heads=1, kv_lens=(400,), block_size=16, steps=2, m_active=9)
    run_blocks(cfg, modes=("losa",))


def test_multi_block_append():
    cfg = wl.config("c5", kv_lens=(200, 90, 64), n_blocks=3, steps=3, topk=4)
    run_blocks(cfg, n_blocks=3)


def test_multi_block_append_fp32_small_pages():
    cfg = wl.config("c1", kv_lens=(100, 7), n_blocks=2, steps=2, topk=3, m_active=3, block_size=24)
    run_blocks(cfg, n_blocks=2)


def test_out_of_range_page_table_is_reported_not_fatal():
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", kv_lens=(256,), block_size=8, steps=2, topk=2, m_active=1)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    inp = w.start_block()
    g.page_table[0, 3] = g.k_pages.shape[0]          # logical page 3 now names the first page outside the pool
    g.run_step(to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk), to_device(inp.m_per_seq))
    assert g.ctx.poll_status() == B.LOSA_ERR_BOUNDS
    assert g.ctx.poll_status() == 0       # cleared by the poll; the context stays usable
    g.page_table[0, 3] = int(w.page_table[0, 3])
    g.step.zero_()
    g.q_prev.zero_()
    g.run_step(to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk), to_device(inp.m_per_seq))
    assert g.ctx.poll_status() == 0
    ref = OracleLayer(w).run_step(inp)
    compare(g.snapshot(), ref, cfg, "after recovery")


def test_prefix_length_beyond_the_page_table_is_reported_not_fatal():
    """kv_len one token past what the page-table row can hold: stages 2 and 3 clamp the page count,
    report LOSA_ERR_BOUNDS and touch nothing outside their rows; a block that does not fit is not
    appended and the length stays as it was."""
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_device, to_host
    cfg = wl.config("c2", kv_lens=(256,), block_size=8, steps=2, topk=2, m_active=2, n_blocks=0)
    assert cfg.max_pages_per_seq == 8
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    i0, i1 = w.start_block(), w.next_step()
    dev = lambda i: (to_device(i.q), to_device(i.k_blk), to_device(i.v_blk), to_device(i.m_per_seq))
    g.run_step(*dev(i0))
    assert g.ctx.poll_status() == 0
    g.kv_len.fill_(8 * 32 + 1)
    g.run_step(*dev(i1))
    assert g.ctx.poll_status() == B.LOSA_ERR_BOUNDS
    snap = g.snapshot()
    assert snap["uc"].max() <= 8 and snap["topk"].max() < 8
    g.kv_len.fill_(256)
    g.finalize_block(*dev(i1)[1:3])                  # 256 + 8 tokens need a ninth page: refused
    assert g.ctx.poll_status() == B.LOSA_ERR_BOUNDS
    assert to_host(g.kv_len).tolist() == [256] and to_host(g.step).tolist() == [0]
    # the context is still good for a whole block (index rows of stable tokens are never written:
    # start them from the fill value the fresh oracle layer starts from)
    g.q_prev.zero_()
    g.topk_pages.fill_(-9)
    o = OracleLayer(w)
    for i in (i0, i1):
        g.run_step(*dev(i))
        assert g.ctx.poll_status() == 0
        compare(g.snapshot(), o.run_step(i), cfg, "after the refused append")


def test_non_finite_rows_never_select_more_than_m_tokens():
    """Inputs must be finite; if they are not, a NaN change score ranks as +inf, so the ranking is
    still a total order and at most m tokens come out (ties on +inf go to the lower index)."""
    import torch
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer
    cfg = wl.config("c1", kv_lens=(64,), block_size=16, steps=2)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    x_prev = torch.zeros((1, 16, 256), device="cuda")
    x_cur = torch.randn((1, 16, 256), device="cuda")
    x_cur[0, 3, 7] = float("nan")
    x_cur[0, 11, 0] = float("inf")
    x_cur[0, 12, 5] = float("nan")
    m = torch.tensor([2], dtype=torch.int32, device="cuda")
    one = torch.ones(1, dtype=torch.int32, device="cuda")
    B.losa_select_active(g.ctx, x_cur, x_prev, 256, m, one, g.active_idx, g.n_active, g.delta)
    assert g.ctx.poll_status() == 0
    assert g.n_active.item() == 2 and g.active_idx[0, :3].tolist() == [3, 11, -1]
    m.fill_(5)
    B.losa_select_active(g.ctx, x_cur, x_prev, 256, m, one, g.active_idx, g.n_active, g.delta)
    assert g.n_active.item() == 5 and set(g.active_idx[0, :5].tolist()) >= {3, 11, 12}


def test_expired_wait_is_reported_and_the_context_stays_usable():
    """The bf16 stage-4 kernel bounds every wait between its warps.  With the bound set to a few
    cycles every thread block gives up at its first wait that is not satisfied at once: it records
    LOSA_ERR_TIMEOUT, lets the copies and tensor-core instructions it had started finish, returns
    its tensor memory and ends normally.  No barrier is starved and nothing hangs; afterwards, with
    the default bound, the same context computes a whole block correctly."""
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", kv_lens=(4096, 1500), steps=3, topk=8, m_active=3)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    steps = w.block_steps()
    dev = lambda i: (to_device(i.q), to_device(i.k_blk), to_device(i.v_blk), to_device(i.m_per_seq))
    g.ctx.set_wait_limit(1)
    g.run_step(*dev(steps[0]))
    assert g.ctx.poll_status() == B.LOSA_ERR_TIMEOUT
    assert g.ctx.poll_status() == 0                       # cleared by the poll
    g.run_step_fused(*dev(steps[0]))                      # the whole-step path reports it the same way
    assert g.ctx.poll_status() == B.LOSA_ERR_TIMEOUT
    g.ctx.set_wait_limit(0)                               # default bound again
    g.step.zero_()
    g.q_prev.zero_()
    g.topk_pages.fill_(-9)
    o = OracleLayer(w)
    for t, i in enumerate(steps):
        g.run_step(*dev(i))
        assert g.ctx.poll_status() == 0
        compare(g.snapshot(), o.run_step(i), cfg, f"after the expired waits, step {t}")


def test_full_size_c3_in_the_benchmark_configuration():
    """The benchmark's workload (ragged 16K/24K/32K/32K batch, 3 active tokens, top-64 pages) at
    full size.  Step 0 (dense): index outputs in full, attention on sampled tokens the oracle
    computes one by one.  Step 1 (LoSA): everything in full — only the active tokens are
    recomputed, so the oracle finishes in seconds."""
    from oracle import oracle as orc
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c3")
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    o = OracleLayer(w)
    inp0, inp1 = w.start_block(), w.next_step()
    N, B = cfg.batch, cfg.block_size
    # ---- step 0
    g.run_step(to_device(inp0.q), to_device(inp0.k_blk), to_device(inp0.v_blk), to_device(inp0.m_per_seq))
    s0 = g.snapshot()
    assert g.ctx.poll_status() == 0
    sh = o.sh
    act, na, _ = orc.select_active(sh, inp0.q, o.q_prev, inp0.m_per_seq, o.step)
    up, uc = orc.page_union(sh, o.topk, act, na, cfg.topk, o.kv_len, o.step)
    for key, ref in (("act", act), ("na", na), ("up", up), ("uc", uc)):
        assert (s0[key] == ref).all(), key
    sample = np.array([0, 13, 31], np.int32)
    act_s = np.full((N, B), -1, np.int32)
    act_s[:, :3] = sample
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    orc.sparse_prefix_attn(sh, inp0.q, o.kv, act_s, np.full(N, 3, np.int32), up, uc, o.o_p, o.lse_p)
    assert_close(s0["o_p"][:, sample], o.o_p[:, sample], cfg.dtype, "step 0 sampled o_p")
    assert_lse_close(s0["lse_p"][:, sample], o.lse_p[:, sample], "step 0 sampled lse_p")
    out, lse = orc.block_attn_merge(sh, inp0.q, inp0.k_blk, inp0.v_blk, o.o_p, o.lse_p)
    assert_close(s0["out"], out, cfg.dtype, "step 0 out")
    assert_lse_close(s0["lse"], lse, "step 0 lse")
    orc.update_prefix_cache(sh, o.kv, o.q_prev, o.step, inp0.q, inp0.k_blk, inp0.v_blk, False)
    # ---- step 1: the oracle state now holds GPU values for the non-sampled tokens (within tolerance)
    g.run_step(to_device(inp1.q), to_device(inp1.k_blk), to_device(inp1.v_blk), to_device(inp1.m_per_seq))
    s1 = g.snapshot()
    assert g.ctx.poll_status() == 0
    ref = o.run_step(inp1)
    for s in range(N):
        assert ref["act"][s, :3].tolist() == inp1.planted[s].tolist()
    compare(s1, ref, cfg, "c3 full size, LoSA step")
    assert 8 * 64 <= ref["uc"].sum() < 26624 // 2


@pytest.mark.parametrize("name,kw", [
    ("c1", dict()),
    ("c2", dict(kv_lens=(2048,), steps=4)),
    ("c2", dict(kv_lens=(5 * 32 + 3, 0, 1, 7 * 32), block_size=12, steps=3, topk=3, m_active=2)),
    ("c5", dict(kv_lens=(200, 90, 64), n_blocks=2, steps=3, topk=4)),
    # in-block attention on the tensor cores: 64 block keys (two row groups of queries), and 48 keys
    # padded to 64 with d = 64 and two heads per KV head
    ("c2", dict(kv_lens=(1000,), block_size=64, steps=3, topk=6, m_active=5)),
    ("c2", dict(n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=16, kv_lens=(700, 333), block_size=48, steps=3,
                topk=5, m_active=3)),
])
def test_whole_step_call_matches_the_oracle(name, kw):
    """losa_denoise_step (one call, in-block attention on a second stream) against the oracle."""
    cfg = wl.config(name, **kw)
    run_blocks(cfg, n_blocks=cfg.n_blocks, fused=True)


def test_model_step_graph_of_several_layers():
    """The benchmark's default launch configuration in small: one CUDA graph holds one denoising step
    of several layers (whole-step calls back to back, each layer with its own pool and state, the
    programmatic launches running on from one layer into the next); a second graph also finalises
    the block.  Every replayed step of every layer is compared with the oracle, over two blocks."""
    import torch
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c2", kv_lens=(1500, 640), steps=3, n_blocks=2, topk=6, m_active=2)
    L = 3
    ws = [wl.Workload(cfg, layer=l) for l in range(L)]
    gpu = [LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len) for w in ws]
    ora = [OracleLayer(w) for w in ws]
    first = [w.start_block() for w in ws]
    bufs = [[to_device(x) for x in (i.q, i.k_blk, i.v_blk, i.m_per_seq)] for i in first]
    for g, b in zip(gpu, bufs):                           # warm-up outside the graph, then rewind
        g.run_step_fused(*b)
    torch.cuda.synchronize()
    for g in gpu:
        g.step.zero_()
    graphs = []
    for fin in (False, True):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            for g, b in zip(gpu, bufs):
                g.run_step_fused(*b)
                if fin:
                    g.finalize_block(b[1], b[2])
        graphs.append(gr)
    for g in gpu:
        g.step.zero_()
    for blk in range(cfg.n_blocks):
        steps = [first] if blk == 0 else [[w.start_block() for w in ws]]
        steps += [[w.next_step() for w in ws] for _ in range(cfg.steps - 1)]
        for t, inps in enumerate(steps):
            last = t == cfg.steps - 1
            for b, i in zip(bufs, inps):
                for dst, src in zip(b, (i.q, i.k_blk, i.v_blk, i.m_per_seq)):
                    dst.copy_(to_device(src))
            graphs[1 if last else 0].replay()             # finalisation leaves the step's results in place
            torch.cuda.synchronize()
            for l, (g, o, i) in enumerate(zip(gpu, ora, inps)):
                assert g.ctx.poll_status() == 0
                snap = g.snapshot()
                ref = o.run_step(i, finalize=last)
                snap["delta"] = ref["delta"]
                compare(snap, ref, cfg, f"layer {l} block {blk} step {t}")
                if last:
                    s2 = g.snapshot()
                    assert (s2["kv_len"] == o.kv_len).all() and (s2["step"] == 0).all()


def test_whole_step_call_in_a_cuda_graph_full_size():
    """The benchmark's launch configuration: the whole-step call captured in a CUDA graph and
    replayed, full-size workload, LoSA step compared with the oracle in full."""
    import torch
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    cfg = wl.config("c3")
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len)
    o = OracleLayer(w)
    inp0, inp1 = w.start_block(), w.next_step()
    q, kb, vb, m = (to_device(x) for x in (inp0.q, inp0.k_blk, inp0.v_blk, inp0.m_per_seq))
    g.run_step_fused(q, kb, vb, m)                       # un-captured first call (step 0, dense)
    torch.cuda.synchronize()
    s0 = g.snapshot()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        g.run_step_fused(q, kb, vb, m)
    for dst, src in ((q, inp1.q), (kb, inp1.k_blk), (vb, inp1.v_blk), (m, inp1.m_per_seq)):
        dst.copy_(to_device(src))
    graph.replay()
    torch.cuda.synchronize()
    s1 = g.snapshot()
    assert g.ctx.poll_status() == 0
    # oracle: step 0 state taken from the GPU (checked elsewhere at full size), step 1 in full
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    o.q_prev[:] = inp0.q
    o.step[:] = 1
    ref = o.run_step(inp1)
    s1["delta"] = ref["delta"]
    compare(s1, ref, cfg, "c3 whole-step call, graph replay")
    assert (s1["step"] == 2).all()



def test_full_size_c5_layer_in_the_benchmark_configuration():
    """One layer of the benchmark's default workload (batch 8 x 32K prefix, Beta(2,18) active
    counts, top-64 pages), generated on the device like the benchmark does, through the whole-step
    call replayed from a CUDA graph, followed by the block finalisation.  The LoSA step is compared
    with the oracle in full; the dense step and the appended block on samples."""
    import torch
    from oracle import oracle as orc
    from paper_2604_12056_b200.layer import LosaLayer
    cfg = wl.config("c5", n_blocks=2)
    dw = wl.DeviceWorkload(cfg, replica=0, layer=17)
    g = LosaLayer(cfg, dw.k_pages, dw.v_pages, dw.page_table, dw.kv_len)
    d0, d1 = dw.start_block(), dw.next_step()
    q, kb, vb, m = d0.q.clone(), d0.k_blk.clone(), d0.v_blk.clone(), d0.m_per_seq.clone()
    g.run_step_fused(q, kb, vb, m)                       # step 0 (dense), un-captured
    torch.cuda.synchronize()
    s0 = g.snapshot()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        g.run_step_fused(q, kb, vb, m)
    for dst, src in ((q, d1.q), (kb, d1.k_blk), (vb, d1.v_blk), (m, d1.m_per_seq)):
        dst.copy_(src)
    graph.replay()
    torch.cuda.synchronize()
    s1 = g.snapshot()
    assert g.ctx.poll_status() == 0
    o = OracleLayer(dw.host_copy())
    h0, h1 = d0.host_copy(), d1.host_copy()
    N, B = cfg.batch, cfg.block_size
    # dense step: two sampled tokens per sequence, one by one on the CPU
    sample = np.array([3, 28], np.int32)
    act_s = np.full((N, B), -1, np.int32)
    act_s[:, :2] = sample
    up = np.full((N, cfg.n_kv_heads, cfg.max_pages_per_seq), -1, np.int32)
    up[:, :, :1024] = np.arange(1024, dtype=np.int32)
    uc = np.full((N, cfg.n_kv_heads), 1024, np.int32)
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    orc.sparse_prefix_attn(o.sh, h0.q, o.kv, act_s, np.full(N, 2, np.int32), up, uc, o.o_p, o.lse_p)
    assert_close(s0["o_p"][:, sample], o.o_p[:, sample], cfg.dtype, "c5 dense step, sampled o_p")
    assert_lse_close(s0["lse_p"][:, sample], o.lse_p[:, sample], "c5 dense step, sampled lse_p")
    # LoSA step in full
    o.q_prev[:] = h0.q
    o.step[:] = 1
    ref = o.run_step(h1)
    m1 = int(h1.m_per_seq[0])
    for s in range(N):
        assert ref["act"][s, :m1].tolist() == sorted(h1.planted[s].tolist())
    s1["delta"] = ref["delta"]
    compare(s1, ref, cfg, "c5 layer, LoSA step from a graph")
    # block finalisation: lengths, and the appended tokens of one sequence / KV head
    g.finalize_block(kb, vb)
    torch.cuda.synchronize()
    s2 = g.snapshot()
    assert (s2["kv_len"] == 32768 + 32).all() and (s2["step"] == 0).all()
    from paper_2604_12056_b200.layer import to_host
    phys = int(to_host(g.page_table)[5, 1024])
    np.testing.assert_array_equal(to_host(g.k_pages[phys, 3]), to_host(kb[5, :, 3]))
    np.testing.assert_array_equal(to_host(g.kmax[phys, 3]), to_host(kb[5, :, 3]).max(0))


def test_full_size_c5_layer_with_pooled_lists():
    """The same layer with one page list per (token, KV head): the LoSA step of the whole-step call
    (bounds from the tensor cores, pooled over the four heads of a KV head, candidates refined with
    exact scores) compared with the oracle in full.  The dense step only supplies the cached state."""
    import torch
    from paper_2604_12056_b200.layer import LosaLayer
    cfg = wl.config("c5", n_blocks=2)
    dw = wl.DeviceWorkload(cfg, replica=0, layer=5)
    g = LosaLayer(cfg, dw.k_pages, dw.v_pages, dw.page_table, dw.kv_len, pooled=True)
    d0, d1 = dw.start_block(), dw.next_step()
    g.run_step_fused(d0.q, d0.k_blk, d0.v_blk, d0.m_per_seq)
    torch.cuda.synchronize()
    s0 = g.snapshot()
    g.run_step_fused(d1.q, d1.k_blk, d1.v_blk, d1.m_per_seq)
    torch.cuda.synchronize()
    s1 = g.snapshot()
    assert g.ctx.poll_status() == 0
    o = OracleLayer(dw.host_copy(), pooled=True)
    h0, h1 = d0.host_copy(), d1.host_copy()
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    o.q_prev[:] = h0.q
    o.step[:] = 1
    ref = o.run_step(h1)
    s1["delta"] = ref["delta"]
    compare(s1, ref, cfg, "c5 layer, pooled lists, LoSA step")
    G = cfg.n_q_heads // cfg.n_kv_heads
    lists = s1["topk"].reshape(cfg.batch, cfg.block_size, cfg.n_kv_heads, G, cfg.topk)
    for s in range(cfg.batch):
        for tok in ref["act"][s, :ref["na"][s]]:
            assert (lists[s, tok] == lists[s, tok, :, :1]).all()      # one list per KV head
    assert ref["uc"].sum() < 8 * 8 * 1024 // 4
