"""Rank plumbing for multi-GPU runs of the benchmark (one process per GPU, torch.distributed).

The path shards by sequence and has no exchange step: every rank runs its own replica of the
workload (weak scaling).  The only collective work is bookkeeping: a barrier around the timed
region and the maximum over ranks of the measured time.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, world_size, local_rank) from the launcher's environment (defaults: single process)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Initialises the default process group when WORLD_SIZE > 1; returns (rank, world, local)."""
    rank, world, local = env_rank()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return rank, world, local


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a host scalar over all ranks (the slowest rank defines the step time)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_of(rank: int) -> int:
    """Workload replica a rank draws (weak scaling: rank r gets its own seeded sequences)."""
    return int(rank)


def shutdown():
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
