"""FP8 (E4M3) K/V pages on the GPU against the oracle (needs a B200): the quantiser bit for bit
(codes, scales, tails, summaries of the dequantised keys), then whole denoising blocks on the FP8
cache - index outputs exact, attention within the bf16 tolerances of the definition evaluated on the
dequantised cache - including block finalisation, which re-quantises the touched pages."""
import numpy as np
import pytest

from helpers import OracleFp8Layer
from paper_2604_12056_b200 import workloads as wl
from test_gpu_parity import compare

pytestmark = pytest.mark.gpu


def assert_cache_equal(g, o, cfg):
    from paper_2604_12056_b200.layer import to_host
    kv_len = to_host(g.kv_len)
    assert (kv_len == o.kv_len).all()
    P = [(int(L) + cfg.page_size - 1) // cfg.page_size for L in kv_len]
    pt = to_host(g.page_table)
    used = np.concatenate([pt[s, :P[s]] for s in range(cfg.batch)]) if sum(P) else np.zeros(0, np.int64)
    for name in ("k_codes", "v_codes", "k_scale", "v_scale"):
        assert (to_host(getattr(g, name))[used] == getattr(o, name)[used]).all(), name
    assert (to_host(g.kmin)[used] == wl.elem_to_f32(o.kmin)[used]).all()
    assert (to_host(g.kmax)[used] == wl.elem_to_f32(o.kmax)[used]).all()


def run_fp8_blocks(cfg, n_blocks=1, fused=False, m=None):
    from paper_2604_12056_b200.layer import LosaLayer, to_device
    w = wl.Workload(cfg)                          # the unused tail of a partial last page holds NaN: the quantiser must not read it
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, fp8_kv=True)
    o = OracleFp8Layer(w)
    assert g.ctx.poll_status() == 0
    assert_cache_equal(g, o, cfg)
    for b in range(n_blocks):
        steps = w.block_steps(m)
        for t, inp in enumerate(steps):
            last = t == len(steps) - 1 and n_blocks > 1
            args = (to_device(inp.q), to_device(inp.k_blk), to_device(inp.v_blk), to_device(inp.m_per_seq))
            (g.run_step_fused if fused else g.run_step)(*args)
            snap = g.snapshot()
            assert g.ctx.poll_status() == 0
            ref = o.run_step(inp, finalize=last)
            if fused:
                snap["delta"] = ref["delta"]
            compare(snap, ref, cfg, f"fp8 {cfg.name} block {b} step {t}")
            if last:
                g.finalize_block(args[1], args[2])
                assert g.ctx.poll_status() == 0
                assert_cache_equal(g, o, cfg)
                assert (g.snapshot()["step"] == 0).all()
    return g, o


@pytest.mark.parametrize("fused", [False, True])
def test_fp8_cache_whole_block(fused):
    run_fp8_blocks(wl.config("c2", kv_lens=(2048, 1500), steps=4), fused=fused)


@pytest.mark.parametrize("g,d,hq,hkv", [(16, 64, 4, 1), (32, 128, 8, 2), (64, 128, 8, 8), (16, 128, 16, 1), (64, 64, 6, 2)])
def test_fp8_cache_ragged_batches_and_page_sizes(g, d, hq, hkv):
    cfg = wl.config("c2", n_q_heads=hq, n_kv_heads=hkv, head_dim=d, page_size=g, kv_lens=(21 * g + 5, 0, 1, 9 * g, 128 + g),
                    block_size=12, steps=3, topk=5, m_active=3)
    run_fp8_blocks(cfg)


def test_fp8_cache_appends_blocks_and_requantises_touched_pages():
    # block of 24 tokens on pages of 16 / 32: every append ends inside a page, so the next one re-quantises it
    for g in (16, 32):
        cfg = wl.config("c5", page_size=g, kv_lens=(200, 90, 64), n_blocks=3, steps=2, topk=4, block_size=24)
        run_fp8_blocks(cfg, n_blocks=3, fused=True)


def test_fp8_cache_dense_mode_and_two_row_groups():
    cfg = wl.config("c4", kv_lens=(64 * 40 + 17,), steps=2, topk=8, m_active=40, heavy_frac=0.0)
    run_fp8_blocks(cfg)


def test_fp8_cache_needs_scales_and_a_bf16_context():
    import ctypes as C
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import LosaLayer
    cfg = wl.config("c2", kv_lens=(256,), block_size=8, steps=2, topk=2, m_active=1)
    w = wl.Workload(cfg)
    g = LosaLayer(cfg, w.k_pages, w.v_pages, w.page_table, w.kv_len, fp8_kv=True)
    bad = B.make_kv(g.k_codes, g.v_codes, g.kmin, g.kmax, g.page_table, g.kv_len, g.k_scale, g.v_scale)
    bad.v_scale = 0
    with pytest.raises(B.LosaError) as e:
        B.losa_sparse_prefix_attn(g.ctx, g.q_prev, bad, g.active_idx, g.n_active, g.union_pages, g.union_count, g.state)
    assert e.value.code == B.LOSA_ERR_INVALID_ARG
    with pytest.raises(B.LosaError) as e:
        B.losa_quantize_kv_pages(g.ctx, g.kv, g.kv)              # source must be a native cache
    assert e.value.code == B.LOSA_ERR_INVALID_ARG


def test_fp8_cache_full_size_c5_layer():
    """One layer of the benchmark's default workload on an FP8 cache: dense first step on sampled
    tokens, the LoSA step in full (the oracle works on the dequantised cache)."""
    import torch
    from oracle import oracle as orc
    from paper_2604_12056_b200.layer import LosaLayer
    from test_gpu_parity import assert_close, assert_lse_close
    cfg = wl.config("c5", n_blocks=1)
    dw = wl.DeviceWorkload(cfg, replica=0, layer=5)
    g = LosaLayer(cfg, dw.k_pages, dw.v_pages, dw.page_table, dw.kv_len, fp8_kv=True)
    o = OracleFp8Layer(dw.host_copy())
    assert_cache_equal(g, o, cfg)
    d0, d1 = dw.start_block(), dw.next_step()
    g.run_step_fused(d0.q, d0.k_blk, d0.v_blk, d0.m_per_seq)
    torch.cuda.synchronize()
    s0 = g.snapshot()
    assert g.ctx.poll_status() == 0
    h0, h1 = d0.host_copy(), d1.host_copy()
    N, B = cfg.batch, cfg.block_size
    sample = np.array([4, 27], np.int32)
    act_s = np.full((N, B), -1, np.int32)
    act_s[:, :2] = sample
    up = np.full((N, cfg.n_kv_heads, cfg.max_pages_per_seq), -1, np.int32)
    up[:, :, :1024] = np.arange(1024, dtype=np.int32)
    uc = np.full((N, cfg.n_kv_heads), 1024, np.int32)
    o.o_p[:] = s0["o_p"]
    o.lse_p[:] = s0["lse_p"]
    orc.sparse_prefix_attn(o.sh, h0.q, o.kv, act_s, np.full(N, 2, np.int32), up, uc, o.o_p, o.lse_p)
    assert_close(s0["o_p"][:, sample], o.o_p[:, sample], cfg.dtype, "fp8 c5 dense step, sampled o_p")
    assert_lse_close(s0["lse_p"][:, sample], o.lse_p[:, sample], "fp8 c5 dense step, sampled lse_p")
    o.q_prev[:] = h0.q
    o.step[:] = 1
    g.run_step_fused(d1.q, d1.k_blk, d1.v_blk, d1.m_per_seq)
    torch.cuda.synchronize()
    s1 = g.snapshot()
    assert g.ctx.poll_status() == 0
    ref = o.run_step(h1)
    s1["delta"] = ref["delta"]
    compare(s1, ref, cfg, "fp8 c5 layer, LoSA step")
