"""The allocation-free stage-1 entry point against the regular one (needs a B200).

Who needs it: programs that may not obtain device memory while they run — a server whose pool was
handed out at start-up, a plug-in under a fixed budget — cannot create the workspace a context
wants.  losa_select_active_static keeps its scratch in a fixed array inside the library instead.
The fixed array is shared by every call on the device and keeps old contents, so the test calls it
twice in a row with different inputs and different active counts and checks both results against
losa_select_active.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2604_12056_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_both(cfg, x_cur, x_prev, m, step):
    from paper_2604_12056_b200 import binding as B
    from paper_2604_12056_b200.layer import to_device, to_host
    N, Bk = cfg.batch, cfg.block_size
    dtype = B.LOSA_BF16 if cfg.dtype == "bf16" else B.LOSA_F32
    ctx = B.Context(N, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, Bk, cfg.page_size,
                    cfg.max_pages_per_seq, dtype, cfg.sm_scale)
    xc, xp = to_device(x_cur), to_device(x_prev)
    md, sd = to_device(m), to_device(step)
    width = x_cur.size // (N * Bk)
    outs = []
    for which in ("regular", "static"):
        act = torch.full((N, Bk), -7, dtype=torch.int32, device="cuda")
        na = torch.full((N,), -7, dtype=torch.int32, device="cuda")
        delta = torch.full((N, Bk), float("nan"), dtype=torch.float32, device="cuda")
        if which == "regular":
            B.losa_select_active(ctx, xc, xp, width, md, sd, act, na, delta)
        else:
            B.losa_select_active_static(ctx.shape, xc, xp, width, md, sd, act, na, delta)
        torch.cuda.synchronize()
        outs.append((to_host(act), to_host(na), to_host(delta)))
    ctx.close()
    return outs


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row(dtype):
    cfg = wl.config("c2", kv_lens=(256, 64, 128), block_size=32, steps=3, dtype=dtype)
    w = wl.Workload(cfg)
    steps = w.block_steps()
    calls = [(steps[1].q, steps[0].q, np.array([3, 1, 5], np.int32), np.array([1, 1, 1], np.int32)),
             (steps[2].q, steps[1].q, np.array([2, 32, 0], np.int32), np.array([2, 0, 2], np.int32))]
    for x_cur, x_prev, m, step in calls:
        (a0, n0, d0), (a1, n1, d1) = run_both(cfg, x_cur, x_prev, m, step)
        assert (a0 == a1).all() and (n0 == n1).all()
        np.testing.assert_allclose(d1, d0, rtol=1e-6, atol=0)
        assert n0.tolist() == [int(mm) if st else 32 for mm, st in zip(m, step)]


def test_static_scratch_entry_point_rejects_oversized_batches():
    from paper_2604_12056_b200 import binding as B
    x = torch.zeros((65, 4, 64), dtype=torch.float32, device="cuda")
    act = torch.zeros((65, 4), dtype=torch.int32, device="cuda")
    na = torch.zeros(65, dtype=torch.int32, device="cuda")
    shape = B.ShapeT(65, 1, 1, 64, 4, 16, 1, B.LOSA_F32, 0.125)
    with pytest.raises(B.LosaError) as e:
        B.losa_select_active_static(shape, x, x, 64, None, None, act, na)
    assert e.value.code == B.LOSA_ERR_UNSUPPORTED
