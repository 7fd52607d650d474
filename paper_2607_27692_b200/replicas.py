"""Rank plumbing for multi-GPU runs of the decode step.

The path shards over (sequence, head) with no exchange, so more GPUs means independent
replicas: one process per GPU, each on its own streams.  Nothing here touches the data
path; it only synchronises the ranks around a timed region and combines their clocks.
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, world_size, local_rank) from the launcher's environment (defaults: single process)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Join the process group when launched with more than one rank; returns the module or None."""
    _, world, _ = rank_info()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kw)
    return dist


def barrier(dist):
    if dist is not None:
        dist.barrier()


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's time: a job of replicas is done when its last replica is."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_cost_per_step(us_per_step_slowest: float, world: int) -> float:
    """N replicas finish N x K steps in the time the slowest needs for K: cost per step of the job."""
    return us_per_step_slowest / max(world, 1)
