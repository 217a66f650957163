"""World-size-2 `gloo` run on CPU of the benchmark's rank plumbing: replicas differ per rank, the
barrier completes, and the reported time is the maximum over ranks."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2604_12056_b200 import dist as D
    from paper_2604_12056_b200 import workloads as wl
    r, w, _ = D.init("gloo")
    assert (r, w) == (rank, world)
    cfg = wl.config("c2", kv_lens=(256,), block_size=8, steps=2, topk=2, m_active=1)
    work = wl.Workload(cfg, replica=D.replica_of(r))
    inp = work.start_block()
    D.barrier()
    t = D.max_over_ranks(10.0 + 5.0 * r)          # rank 1 is "slower"
    np.save(os.path.join(out_dir, f"r{r}.npy"),
            np.array([t, float(np.asarray(inp.q, np.float64).sum()), float(work.page_table.sum())]))
    D.shutdown()


def test_two_gloo_ranks_weak_scaling_bookkeeping(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    a, b = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    assert a[0] == b[0] == 15.0                   # max over ranks, identical on every rank
    assert a[1] != b[1]                           # different replicas draw different inputs
    assert a[2] == b[2]                           # same pool size, so the same sum of page ids


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    from paper_2604_12056_b200 import dist as D
    assert D.env_rank() == (0, 1, 0)
    assert D.max_over_ranks(3.5) == 3.5
    D.barrier()
