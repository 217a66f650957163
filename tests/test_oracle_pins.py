"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test names the passage it pins.  The references here are brute force from the definitions
(numpy fp64, torch SDPA fp64, numpy argsort / unique), never the oracle's own code.
"""
import os

import numpy as np
import pytest

from helpers import Problem, softmax_attention, torch_sdpa
from oracle import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def dense_step(pb: Problem, m=None, k=None, step0=True):
    """Runs stages 1-5 of the oracle on pb (state freshly allocated)."""
    sh = pb.sh
    N, B, H, d = sh.batch, sh.block_size, sh.n_q_heads, sh.head_dim
    orc.build_page_summaries(sh, pb.kv)
    step = np.zeros(N, np.int32) if step0 else np.ones(N, np.int32)
    mm = None if m is None else np.full(N, m, np.int32)
    act, na, _ = orc.select_active(sh, pb.q, pb.q_prev if hasattr(pb, "q_prev") else pb.q, mm, step)
    kk = k if k is not None else sh.max_pages_per_seq
    topk, _ = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, kk, step)
    up, uc = orc.page_union(sh, topk, act, na, kk, pb.kv_len, step)
    o_p = np.full((N, B, H, d), 7.0)
    lse_p = np.full((N, B, H), 7.0)
    orc.sparse_prefix_attn(sh, pb.q, pb.kv, act, na, up, uc, o_p, lse_p)
    out, lse = orc.block_attn_merge(sh, pb.q, pb.k_blk, pb.v_blk, o_p, lse_p)
    return dict(act=act, na=na, topk=topk, up=up, uc=uc, o_p=o_p, lse_p=lse_p, out=out, lse=lse)


def brute_full(pb: Problem, s, i, h):
    """Section 2.1 full-attention equation for one query: softmax over [K_p, K_b]."""
    G = pb.sh.n_q_heads // pb.sh.n_kv_heads
    kh = h // G
    K = np.concatenate([pb.K[s][:, kh], pb.f(pb.k_blk)[s, :, kh]], 0)
    V = np.concatenate([pb.V[s][:, kh], pb.f(pb.v_blk)[s, :, kh]], 0)
    return K, V, pb.f(pb.q)[s, i, h]


# --- I1: every token active and every page selected  ==  dense attention (Section 2.1) ----------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["step0", "topk_all"])
def test_all_active_all_pages_is_dense_attention(dtype, mode):
    pb = Problem(1, N=2, Hq=4, Hkv=2, d=16, B=5, g=4, kv_lens=(19, 8), dtype=dtype)
    r = dense_step(pb, step0=(mode == "step0"))
    sh = pb.sh
    for s in range(sh.batch):
        for i in range(sh.block_size):
            for h in range(sh.n_q_heads):
                K, V, q = brute_full(pb, s, i, h)
                o, lse = softmax_attention(q, K, V, sh.sm_scale)
                np.testing.assert_allclose(r["out"][s, i, h], o, rtol=0, atol=1e-12)
                np.testing.assert_allclose(r["lse"][s, i, h], lse, rtol=0, atol=1e-12)
                np.testing.assert_allclose(r["out"][s, i, h], torch_sdpa(q, K, V, sh.sm_scale),
                                           rtol=0, atol=1e-12)


# --- I2: LSE merge of two key sets == softmax over their concatenation (Section 2.2) -------------
@pytest.mark.parametrize("scale", [1.0, 30.0])
@pytest.mark.parametrize("kv_len", [0, 1, 7, 16])
def test_lse_merge_equals_concatenation(scale, kv_len):
    pb = Problem(2 + kv_len, N=1, Hq=2, Hkv=1, d=16, B=3, g=4, kv_lens=(kv_len,), scale=scale)
    r = dense_step(pb)
    for i in range(3):
        for h in range(2):
            K, V, q = brute_full(pb, 0, i, h)
            o, lse = softmax_attention(q, K, V, pb.sh.sm_scale)
            np.testing.assert_allclose(r["out"][0, i, h], o, rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(r["lse"][0, i, h], lse, rtol=1e-12, atol=1e-12)
            # the prefix part alone is attention over the prefix keys only
            op, lp = softmax_attention(q, pb.K[0][:, 0], pb.V[0][:, 0], pb.sh.sm_scale)
            np.testing.assert_allclose(r["o_p"][0, i, h], op, rtol=1e-12, atol=1e-12)
            if kv_len == 0:
                assert r["lse_p"][0, i, h] == -np.inf
            else:
                np.testing.assert_allclose(r["lse_p"][0, i, h], lp, rtol=1e-12, atol=1e-12)


# --- I3: reuse rule — stable tokens keep (o_p, L_p) bit for bit (Section 4.2) ---------------------
def test_stable_tokens_reuse_cached_statistics_exactly():
    pb = Problem(3, N=1, Hq=4, Hkv=2, d=16, B=6, g=4, kv_lens=(23,))
    sh = pb.sh
    r0 = dense_step(pb)
    o_p, lse_p = r0["o_p"].copy(), r0["lse_p"].copy()
    q_prev = pb.q.copy()
    q = pb.q.copy()
    q[0, 1] = pb.rand_elem(q[0, 1].shape)
    q[0, 4] = pb.rand_elem(q[0, 4].shape)
    step = np.ones(1, np.int32)
    act, na, delta = orc.select_active(sh, q, q_prev, np.array([2], np.int32), step)
    assert act[0].tolist() == [1, 4, -1, -1, -1, -1] and na[0] == 2
    assert (delta[0, [0, 2, 3, 5]] == 0).all()
    topk, _ = orc.page_scores_topk(sh, q, pb.kv, act, na, 2, step)
    up, uc = orc.page_union(sh, topk, act, na, 2, pb.kv_len, step)
    orc.sparse_prefix_attn(sh, q, pb.kv, act, na, up, uc, o_p, lse_p)
    stable = [0, 2, 3, 5]
    assert (o_p[0, stable] == r0["o_p"][0, stable]).all()
    assert (lse_p[0, stable] == r0["lse_p"][0, stable]).all()
    assert not (o_p[0, [1, 4]] == r0["o_p"][0, [1, 4]]).any()
    # unchanged block K/V and bit-identical query => bit-identical final output
    out, _ = orc.block_attn_merge(sh, q, pb.k_blk, pb.v_blk, o_p, lse_p)
    assert (out[0, stable] == r0["out"][0, stable]).all()


# --- I9 / I10: active queries attend over the shared union (Section 4.2) ---------------------------
def test_union_attention_equals_dense_on_the_kept_pages():
    pb = Problem(4, N=1, Hq=4, Hkv=2, d=16, B=4, g=4, kv_lens=(30,))
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    act = np.array([[0, 2, -1, -1]], np.int32)
    na = np.array([2], np.int32)
    up = np.full((1, 2, sh.max_pages_per_seq), -1, np.int32)
    up[0, 0, :3] = [1, 4, 7]          # page 7 is partial: tokens 28, 29
    up[0, 1, :2] = [0, 5]
    uc = np.array([[3, 2]], np.int32)
    o_p = np.full((1, 4, 4, 16), 3.0)
    lse_p = np.full((1, 4, 4), 3.0)
    orc.sparse_prefix_attn(sh, pb.q, pb.kv, act, na, up, uc, o_p, lse_p)
    for i in (0, 2):
        for h in range(4):
            kh = h // 2
            toks = np.concatenate([np.arange(p * 4, min(30, p * 4 + 4)) for p in up[0, kh, :uc[0, kh]]])
            o, lse = softmax_attention(pb.f(pb.q)[0, i, h], pb.K[0][toks, kh], pb.V[0][toks, kh], sh.sm_scale)
            np.testing.assert_allclose(o_p[0, i, h], o, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(lse_p[0, i, h], lse, rtol=1e-12)
    assert (o_p[0, [1, 3]] == 3.0).all() and (lse_p[0, [1, 3]] == 3.0).all()


def test_budget_covering_all_pages_gives_dense_prefix_for_active_only():
    pb = Problem(5, N=1, Hq=2, Hkv=1, d=16, B=4, g=4, kv_lens=(13,))
    sh = pb.sh
    pb.q_prev = pb.q.copy()
    pb.q[0, 3] = pb.rand_elem(pb.q[0, 3].shape)
    r = dense_step(pb, m=1, k=99, step0=False)
    assert r["act"][0].tolist() == [3, -1, -1, -1]
    assert r["uc"][0, 0] == 4 and r["up"][0, 0, :4].tolist() == [0, 1, 2, 3]
    for h in range(2):
        o, lse = softmax_attention(pb.f(pb.q)[0, 3, h], pb.K[0][:, 0], pb.V[0][:, 0], sh.sm_scale)
        np.testing.assert_allclose(r["o_p"][0, 3, h], o, rtol=1e-12, atol=1e-13)
    assert (r["o_p"][0, :3] == 7.0).all()


# --- I5 / I6: the page score is an upper bound; at page size 1 it is the dot product (Section 2.3) --
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_page_score_is_an_upper_bound(dtype):
    pb = Problem(6, N=1, Hq=4, Hkv=2, d=32, B=3, g=8, kv_lens=(61,), dtype=dtype)
    orc.build_page_summaries(pb.sh, pb.kv)
    for i in range(3):
        for h in range(4):
            u32, u64 = orc.page_scores_one(pb.sh, pb.q, pb.kv, 0, i, h)
            q = pb.f(pb.q)[0, i, h]
            for p in range(pb.pages(0)):
                toks = np.arange(p * 8, min(61, p * 8 + 8))
                dots = pb.K[0][toks, h // 2].astype(np.float64) @ q
                assert u64[p] >= dots.max() - 1e-12
                # tight: some key box corner attains it, so it cannot exceed sum |q| * max|k|
                assert u64[p] <= (np.abs(q) * np.abs(pb.K[0][toks, h // 2]).max(0)).sum() + 1e-12
                assert abs(float(u32[p]) - u64[p]) <= 32 * 2.0 ** -23 * np.abs(q[None] * pb.K[0][toks, h // 2]).max(0).sum() + 1e-30


def test_page_size_one_selects_exact_topk_keys():
    pb = Problem(7, N=1, Hq=2, Hkv=1, d=16, B=2, g=1, kv_lens=(40,), extra_pages=0)
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    act = np.array([[0, 1]], np.int32)
    na = np.array([2], np.int32)
    topk, sc = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, 5)
    for i in range(2):
        for h in range(2):
            u32, u64 = orc.page_scores_one(sh, pb.q, pb.kv, 0, i, h)
            dots = pb.K[0][:, 0].astype(np.float64) @ pb.f(pb.q)[0, i, h]
            np.testing.assert_allclose(u64, dots, rtol=0, atol=1e-13)   # equality at g = 1
            want = np.argsort(-dots, kind="stable")[:5]
            assert topk[0, i, h].tolist() == want.tolist()
            np.testing.assert_allclose(sc[0, i, h], dots[want], rtol=1e-5, atol=1e-6)


def test_topk_order_ties_and_padding():
    # identical pages => identical scores => ties resolved by lower page index; k > P pads with -1
    pb = Problem(8, N=1, Hq=1, Hkv=1, d=16, B=1, g=2, kv_lens=(12,), extra_pages=1, shuffle=True)
    sh = pb.sh
    for p in range(1, 6):                       # copy page 0 into every page
        pb.k_pages[pb.page_table[0, p]] = pb.k_pages[pb.page_table[0, 0]]
    orc.build_page_summaries(sh, pb.kv)
    act, na = np.array([[0]], np.int32), np.array([1], np.int32)
    topk, sc = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, 8)
    assert topk[0, 0, 0].tolist() == [0, 1, 2, 3, 4, 5, -1, -1]
    assert len(set(sc[0, 0, 0, :6].tolist())) == 1 and np.isnan(sc[0, 0, 0, 6:]).all()
    topk3, _ = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, 3)
    assert topk3[0, 0, 0].tolist() == [0, 1, 2]


@pytest.mark.parametrize("d", [64, 128])
def test_fixed_order_fp32_score_matches_its_specification(d):
    """The interface fixes the fp32 summation order; re-derive it in exact rational arithmetic with
    explicit roundings, for both head dimensions (d / 8 runs, butterfly offsets d / 16 .. 1)."""
    pb = Problem(9, N=1, Hq=2, Hkv=1, d=d, B=1, g=4, kv_lens=(64,))
    orc.build_page_summaries(pb.sh, pb.kv)
    u32, _ = orc.page_scores_one(pb.sh, pb.q, pb.kv, 0, 0, 1)
    q = pb.q[0, 0, 1].astype(np.float32)
    from fractions import Fraction

    def round_f32(x: Fraction) -> np.float32:
        """Exact rational -> nearest float32, ties to even (no double rounding)."""
        f = np.float32(float(x))                      # float(Fraction) is correctly rounded to fp64
        cands = {f, np.nextafter(f, np.float32(np.inf)), np.nextafter(f, np.float32(-np.inf))}
        best = min(cands, key=lambda c: (abs(Fraction(float(c)) - x), int(np.float32(c).view(np.uint32)) & 1))
        return np.float32(best)

    def fma32(a, b, c):
        return round_f32(Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c)))

    for p in range(16):
        ph = pb.page_table[0, p]
        lo, hi = pb.kmin[ph, 0], pb.kmax[ph, 0]
        runs = d // 8
        c = np.zeros(runs, np.float32)
        for r in range(runs):
            acc = np.float32(0.0)
            for jj in range(8):
                j = 8 * r + jj
                acc = fma32(max(q[j], np.float32(0)), hi[j], acc)
                acc = fma32(min(q[j], np.float32(0)), lo[j], acc)
            c[r] = acc
        off = runs // 2
        while off >= 1:
            c = np.array([np.float32(c[i] + c[i ^ off]) for i in range(runs)], np.float32)
            off //= 2
        assert np.float32(c[0] + np.float32(0.0)).tobytes() == u32[p].tobytes()


# --- selector variant: one list per (token, KV head), pooled over the G heads (Section 2.3 leaves the selector open)
def test_pooled_selector_worked_example():
    # pages of one token, two heads sharing one KV head; q0 = e0, q1 = e1, keys (a_p, b_p, 0, ...):
    # head 0 scores a_p, head 1 scores b_p, the pooled score is max(a_p, b_p) - all exact in fp32
    pb = Problem(21, N=1, Hq=2, Hkv=1, d=16, B=1, g=1, kv_lens=(6,), extra_pages=0, shuffle=True)
    keys = [(3, 0), (1, 5), (2, 2), (5, 1), (0, 4), (4, 4)]
    pb.q[:] = 0
    pb.q[0, 0, 0, 0] = 1.0
    pb.q[0, 0, 1, 1] = 1.0
    for p, (a, b) in enumerate(keys):
        row = np.zeros(16, np.float32)
        row[0], row[1] = a, b
        pb.k_pages[pb.page_table[0, p], 0, 0] = row
    orc.build_page_summaries(pb.sh, pb.kv)
    act, na = np.array([[0]], np.int32), np.array([1], np.int32)
    per_head, _ = orc.page_scores_topk(pb.sh, pb.q, pb.kv, act, na, 4)
    assert per_head[0, 0, 0].tolist() == [3, 5, 0, 2]          # a_p: 5, 4, 3, 2
    assert per_head[0, 0, 1].tolist() == [1, 4, 5, 2]          # b_p: 5, 4, 4 (tie: lower page first), 2
    pooled, sc = orc.page_scores_topk_pooled(pb.sh, pb.q, pb.kv, act, na, 4)
    for h in range(2):
        assert pooled[0, 0, h].tolist() == [1, 3, 4, 5]        # max: 5, 5 (pages 1, 3), 4, 4 (pages 4, 5)
        assert sc[0, 0, h].tolist() == [5.0, 5.0, 4.0, 4.0]
    wide, _ = orc.page_scores_topk_pooled(pb.sh, pb.q, pb.kv, act, na, 8)
    assert wide[0, 0, 1].tolist() == [1, 3, 4, 5, 0, 2, -1, -1]


def test_pooled_selector_brute_force_and_invariants():
    pb = Problem(22, N=2, Hq=8, Hkv=2, d=32, B=4, g=4, kv_lens=(90, 37))
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    act = np.array([[1, 3, -1, -1], [0, 2, 3, -1]], np.int32)
    na = np.array([2, 3], np.int32)
    k = 5
    pooled, sc = orc.page_scores_topk_pooled(sh, pb.q, pb.kv, act, na, k)
    per_head, _ = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, k)
    G = 4
    for s in range(2):
        P = pb.pages(s)
        for tok in act[s, :na[s]]:
            for kh in range(2):
                rows = np.stack([orc.page_scores_one(sh, pb.q, pb.kv, s, int(tok), kh * G + gi)[0] for gi in range(G)])
                best = rows.max(axis=0)                                   # fp32 values, exact maximum
                want = np.argsort(-best, kind="stable")[:k]                # ties: lower page first
                for gi in range(G):
                    assert pooled[s, tok, kh * G + gi].tolist() == want.tolist()
                    assert sc[s, tok, kh * G + gi].tobytes() == best[want].tobytes()
                # every pooled page is in the list of the head that attains its score (no ties in this data)
                lists = {int(p) for gi in range(G) for p in per_head[s, tok, kh * G + gi]}
                assert set(want.tolist()) <= lists
    # untouched rows keep the fill value
    assert (pooled[0, 0] == -9).all() and (pooled[1, 1] == -9).all()
    # the union can only shrink, and is bounded by (active tokens) * k per KV head
    up_h, uc_h = orc.page_union(sh, per_head, act, na, k, pb.kv_len)
    up_p, uc_p = orc.page_union(sh, pooled, act, na, k, pb.kv_len)
    for s in range(2):
        for kh in range(2):
            a, b = set(up_p[s, kh, :uc_p[s, kh]].tolist()), set(up_h[s, kh, :uc_h[s, kh]].tolist())
            assert a <= b and k <= len(a) <= na[s] * k


def test_pooled_selector_without_grouping_is_the_per_head_selector():
    pb = Problem(23, N=1, Hq=3, Hkv=3, d=16, B=3, g=2, kv_lens=(33,))
    orc.build_page_summaries(pb.sh, pb.kv)
    act, na = np.array([[0, 2, -1]], np.int32), np.array([2], np.int32)
    a, sa = orc.page_scores_topk(pb.sh, pb.q, pb.kv, act, na, 6)
    b, sb = orc.page_scores_topk_pooled(pb.sh, pb.q, pb.kv, act, na, 6)
    assert (a == b).all() and sa.tobytes() == sb.tobytes()


# --- I4: union-size inequalities (Section 4.4; worst case of Section 3.1) --------------------------
def test_union_inequalities_and_subset():
    pb = Problem(10, N=2, Hq=4, Hkv=2, d=16, B=8, g=4, kv_lens=(90, 57))
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    k, G = 3, 2
    step = np.ones(2, np.int32)
    q_prev = pb.q.copy()
    q = pb.q.copy()
    q[:, [2, 5]] = pb.rand_elem(q[:, [2, 5]].shape)
    actA, naA, _ = orc.select_active(sh, q, q_prev, np.array([2, 2], np.int32), step)
    actB, naB, _ = orc.select_active(sh, q, q_prev, None, step)
    assert naB.tolist() == [8, 8]
    tA, _ = orc.page_scores_topk(sh, q, pb.kv, actA, naA, k, step)
    tB, _ = orc.page_scores_topk(sh, q, pb.kv, actB, naB, k, step)
    assert (tA[:, [2, 5]] == tB[:, [2, 5]]).all()       # selection of a query does not depend on A
    uA, cA = orc.page_union(sh, tA, actA, naA, k, pb.kv_len, step)
    uB, cB = orc.page_union(sh, tB, actB, naB, k, pb.kv_len, step)
    for s in range(2):
        P = pb.pages(s)
        for kh in range(2):
            a = uA[s, kh, :cA[s, kh]]
            b = uB[s, kh, :cB[s, kh]]
            assert min(k, P) <= cA[s, kh] <= min(P, 2 * G * k)
            assert cA[s, kh] <= cB[s, kh] <= min(P, 8 * G * k)
            assert set(a.tolist()) <= set(b.tolist())
            assert (np.diff(a) > 0).all() and (np.diff(b) > 0).all()
            want = np.unique(tA[s, [2, 5]][:, kh * G:(kh + 1) * G].ravel())
            assert a.tolist() == want[want >= 0].tolist()          # textbook union (numpy.unique)
            assert (uA[s, kh, cA[s, kh]:] == -1).all()


# --- I7: Eq. 1 and the pruning rule (Section 3.2, Section 4.1) --------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_locality_score_and_ranking(dtype):
    pb = Problem(11, N=2, Hq=4, Hkv=2, d=16, B=7, g=4, kv_lens=(8, 8), dtype=dtype)
    sh = pb.sh
    x0 = pb.rand_elem((2, 7, 40))
    x1 = x0.copy()
    act, na, delta = orc.select_active(sh, x1, x0, np.array([3, 0], np.int32), np.ones(2, np.int32))
    assert (delta == 0).all() and act[0].tolist() == [0, 1, 2, -1, -1, -1, -1] and na.tolist() == [3, 0]
    x1[0, 5] = pb.rand_elem((40,))
    x1[0, 2] = pb.rand_elem((40,), scale=3.0)
    x1[1, 6] = pb.rand_elem((40,))
    act, na, delta = orc.select_active(sh, x1, x0, np.array([2, 1], np.int32), np.ones(2, np.int32))
    want = ((pb.f(x1) - pb.f(x0)) ** 2).mean(-1)
    np.testing.assert_allclose(delta, want, rtol=1e-13, atol=0)
    assert act[0].tolist() == [2, 5, -1, -1, -1, -1, -1] and act[1].tolist() == [6, -1, -1, -1, -1, -1, -1]
    order = np.argsort(-want[0], kind="stable")[:4]
    act4, _, _ = orc.select_active(sh, x1, x0, np.array([4, 4], np.int32), np.ones(2, np.int32))
    assert act4[0, :4].tolist() == sorted(order.tolist())
    # step 0 or no m: everything active (Initialization Workflow, Section 4.2)
    act0, na0, _ = orc.select_active(sh, x1, x0, np.array([2, 1], np.int32), np.array([0, 1], np.int32))
    assert na0.tolist() == [7, 1] and act0[0].tolist() == list(range(7))
    actn, nan_, _ = orc.select_active(sh, x1, x0, None, None)
    assert nan_.tolist() == [7, 7]


# --- I7b: threshold variant of the pruning rule (appendix heat maps, tau = 0.5) --------------------
def test_threshold_pruning_rule():
    # a worked example with exact arithmetic: one changed element per token gives Delta_i = c_i^2 / w
    pb = Problem(12, N=2, Hq=4, Hkv=2, d=16, B=6, g=4, kv_lens=(8, 8), dtype="f32")
    sh, w = pb.sh, 16
    x0 = np.zeros((2, 6, w), np.float32)
    x1 = x0.copy()
    amps = np.array([1.0, 4.0, 2.0, 0.0, 2.0, 1.0], np.float32)          # squares 1 16 4 0 4 1: total 26
    x1[0, np.arange(6), 0] = amps
    x1[1] = 0.0                                                          # nothing changed: no active token
    one = np.ones(2, np.int32)
    act, na, delta = orc.select_active_tau(sh, x1, x0, 0.5, None, one)
    np.testing.assert_array_equal(delta[0] * w, amps.astype(np.float64) ** 2)
    assert na.tolist() == [1, 0] and act[0, 0] == 1                      # 16 >= 13
    act, na, _ = orc.select_active_tau(sh, x1, x0, 16.0 / 26.0 + 1e-9, None, one)
    assert na[0] == 2 and act[0, :2].tolist() == [1, 2]                  # tie 4 = 4: the lower index first
    act, na, _ = orc.select_active_tau(sh, x1, x0, 24.0 / 26.0, None, one)
    assert na[0] == 3 and act[0, :3].tolist() == [1, 2, 4]               # 16 + 4 + 4 = 24 reaches 24 exactly
    act, na, _ = orc.select_active_tau(sh, x1, x0, 1.0, None, one)
    assert na[0] == 5 and act[0, :5].tolist() == [0, 1, 2, 4, 5]         # the unchanged token is never needed
    act, na, _ = orc.select_active_tau(sh, x1, x0, 1.0, np.array([2, 2], np.int32), one)
    assert na.tolist() == [2, 0] and act[0, :2].tolist() == [1, 2]       # capped
    act, na, _ = orc.select_active_tau(sh, x1, x0, 0.5, None, np.zeros(2, np.int32))
    assert na.tolist() == [6, 6]                                         # first step of a block: everything
    # against numpy on random data: sort, cumulative sum, first index reaching tau * total
    rng = np.random.default_rng(5)
    pb2 = Problem(13, N=3, Hq=4, Hkv=2, d=16, B=16, g=4, kv_lens=(8, 8, 8), dtype="bf16")
    y0 = pb2.rand_elem((3, 16, 24))
    y1 = y0.copy()
    for s_ in range(3):
        for t in rng.choice(16, size=5, replace=False):
            y1[s_, t] = pb2.rand_elem((24,), scale=float(rng.uniform(0.2, 3.0)))
    for tau in (0.25, 0.5, 0.9):
        act, na, delta = orc.select_active_tau(pb2.sh, y1, y0, tau, None, np.ones(3, np.int32))
        for s_ in range(3):
            order = np.argsort(-delta[s_], kind="stable")
            cum = np.cumsum(delta[s_][order])
            m = int(np.searchsorted(cum, tau * cum[-1], side="left")) + 1
            assert abs(cum[m - 1] - tau * cum[-1]) > 1e-9 * cum[-1]      # the case is not a near-tie
            assert na[s_] == m and act[s_, :m].tolist() == sorted(order[:m].tolist())


# --- I8: results do not depend on where pages live physically --------------------------------------
def test_physical_page_permutation_invariance():
    a = Problem(12, N=2, Hq=4, Hkv=2, d=16, B=4, g=4, kv_lens=(27, 14), shuffle=True)
    b = Problem(12, N=2, Hq=4, Hkv=2, d=16, B=4, g=4, kv_lens=(27, 14), shuffle=False)
    # same seed draws a different stream once the permutation is skipped, so copy the data over
    b.q, b.k_blk, b.v_blk = a.q.copy(), a.k_blk.copy(), a.v_blk.copy()
    for s in range(2):
        for p in range(a.pages(s)):
            b.k_pages[b.page_table[s, p]] = a.k_pages[a.page_table[s, p]]
            b.v_pages[b.page_table[s, p]] = a.v_pages[a.page_table[s, p]]
    for pb in (a, b):
        pb.q_prev = pb.q.copy()
    a.q[:, 1] = a.rand_elem(a.q[:, 1].shape)
    b.q[:, 1] = a.q[:, 1]
    ra = dense_step(a, m=1, k=2, step0=False)
    rb = dense_step(b, m=1, k=2, step0=False)
    for key in ("act", "topk", "up", "uc"):
        assert (ra[key] == rb[key]).all(), key
    assert (ra["o_p"][:, 1] == rb["o_p"][:, 1]).all() and (ra["out"] == rb["out"]).all()


# --- Section 2.1 / 2.3: the cache grows by the finalised block; summaries are min / max -------------
def test_finalize_appends_block_and_refreshes_summaries():
    pb = Problem(13, N=2, Hq=2, Hkv=2, d=16, B=5, g=4, kv_lens=(10, 3), extra_pages=3)
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    q_prev = np.zeros_like(pb.q)
    step = np.array([3, 3], np.int32)
    orc.update_prefix_cache(sh, pb.kv, q_prev, step, pb.q, pb.k_blk, pb.v_blk, False)
    assert (q_prev == pb.q).all() and step.tolist() == [4, 4]
    orc.update_prefix_cache(sh, pb.kv, q_prev, step, pb.q, pb.k_blk, pb.v_blk, True)
    assert pb.kv_len.tolist() == [15, 8] and step.tolist() == [0, 0]
    for s in range(2):
        Kfull = np.concatenate([pb.K[s], pb.f(pb.k_blk)[s]], 0)
        Vfull = np.concatenate([pb.V[s], pb.f(pb.v_blk)[s]], 0)
        for t in range(int(pb.kv_len[s])):
            ph = pb.page_table[s, t // 4]
            assert (pb.f(pb.k_pages)[ph, :, t % 4] == Kfull[t]).all()
            assert (pb.f(pb.v_pages)[ph, :, t % 4] == Vfull[t]).all()
        for p in range(pb.pages(s)):
            ph = pb.page_table[s, p]
            rows = Kfull[p * 4:min(int(pb.kv_len[s]), p * 4 + 4)]
            assert (pb.f(pb.kmin)[ph] == rows.min(0)).all() and (pb.f(pb.kmax)[ph] == rows.max(0)).all()
    # a dense step on the grown cache equals brute force over the grown prefix
    pb.K = [np.concatenate([pb.K[s], pb.f(pb.k_blk)[s]], 0) for s in range(2)]
    pb.V = [np.concatenate([pb.V[s], pb.f(pb.v_blk)[s]], 0) for s in range(2)]
    r = dense_step(pb)
    K, V, q = brute_full(pb, 1, 2, 1)
    o, _ = softmax_attention(q, K, V, sh.sm_scale)
    np.testing.assert_allclose(r["out"][1, 2, 1], o, rtol=0, atol=1e-12)


# --- I11: what the paper prints about sizes ---------------------------------------------------------
def test_paper_stated_sizes():
    facts = {}
    with open(os.path.join(GOLDEN, "paper_facts.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                facts[k.strip()] = int(v)
    B, d = facts["B"], facts["d"]
    assert B * (d + 1) == facts["state_scalars_per_head"]
    pb = Problem(14, N=1, Hq=1, Hkv=1, d=16, B=4, g=4, kv_lens=(4,))
    r = dense_step(pb)
    assert r["o_p"][0, :, 0].size + r["lse_p"][0, :, 0].size == 4 * (16 + 1)
    # worst case of the union (Section 3.1): min(L, B k) positions
    L, k = facts["example_L"], facts["example_k"]
    assert min(L, B * k) == facts["example_union_worst"]


# --- relaxed validity rule for selectors with their own arithmetic (Section 2.3 leaves the selector open)
def test_relaxed_list_rule_accepts_the_exact_lists_and_rejects_worse_ones():
    pb = Problem(31, N=2, Hq=4, Hkv=2, d=32, B=3, g=4, kv_lens=(90, 37))
    sh = pb.sh
    orc.build_page_summaries(sh, pb.kv)
    act = np.array([[0, 2, -1], [1, -1, -1]], np.int32)
    na = np.array([2, 1], np.int32)
    k = 5
    topk, _ = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, k)
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, topk, 0.0) == 0          # exact lists pass with no slack
    shuffled = topk.copy()
    shuffled[0, 0, 1] = topk[0, 0, 1][::-1]                                           # order is not part of the rule
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, shuffled, 0.0) == 0
    # replace the weakest chosen page of one list by the worst page of all: invalid at any small slack
    _, u64 = orc.page_scores_one(sh, pb.q, pb.kv, 0, 2, 3)
    worst = int(np.argmin(u64))
    bad = topk.copy()
    assert worst not in bad[0, 2, 3].tolist()
    bad[0, 2, 3, k - 1] = worst
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, bad, 1e-6) == 1
    # ... but valid once the slack covers the gap (brute force of the rule's own inequality)
    kth = np.sort(u64)[::-1][k - 1]
    lo, hi = pb.f(pb.kmin), pb.f(pb.kmax)
    qv = pb.f(pb.q)[0, 2, 3].astype(np.float64)
    smax = 0.0
    for p in range(pb.pages(0)):
        ph = pb.page_table[0, p]
        t = np.maximum(qv * lo[ph, 1].astype(np.float64), qv * hi[ph, 1].astype(np.float64))
        smax = max(smax, np.abs(t).sum())
    need = (kth - u64[worst]) / smax
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, bad, need * 1.01) == 0
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, bad, need * 0.99) == 1
    # structural violations: a repeated page, an out-of-range page, a missing entry, wrong padding
    for edit in (lambda t: t.__setitem__((1, 1, 0, 1), t[1, 1, 0, 0]), lambda t: t.__setitem__((1, 1, 0, 0), 10),
                 lambda t: t.__setitem__((1, 1, 0, 4), -1)):
        t2 = topk.copy()
        edit(t2)
        assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, k, t2, 1.0) == 1
    wide, _ = orc.page_scores_topk(sh, pb.q, pb.kv, act, na, 12)                        # k > P for sequence 1 (10 pages)
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, 12, wide, 0.0) == 0
    wide[1, 1, 2, 11] = 3
    assert orc.check_topk_relaxed(sh, pb.q, pb.kv, act, na, 12, wide, 1.0) == 1
