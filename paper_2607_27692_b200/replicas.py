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


def under_launcher() -> bool:
    """True when a launcher (torchrun or ``spawn`` below) already set this process's rank."""
    return "RANK" in os.environ and "WORLD_SIZE" in os.environ


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn(argv, n: int, extra_env=None, timeout=None) -> int:
    """Start ``n`` replicas of the command ``argv`` on this node, one process per GPU.

    Rank i gets RANK = LOCAL_RANK = i, WORLD_SIZE = n and a rendezvous on 127.0.0.1 at a free
    port.  Rank 0 inherits stdout (it prints the job's line); the other ranks' stdout is
    dropped, every rank's stderr is inherited.  Returns the first non-zero exit code, or 0;
    if a rank fails the others are ended (they would wait in a collective for ever).
    """
    import subprocess
    import time
    port = free_port()
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen(argv, env=env, stdout=None if rank == 0 else subprocess.DEVNULL))
    deadline = None if timeout is None else time.time() + timeout
    rc = 0
    pending = set(range(n))
    while pending:
        for i in sorted(pending):
            code = procs[i].poll()
            if code is not None:
                pending.discard(i)
                if code != 0 and rc == 0:
                    rc = code
        if rc != 0 or (deadline is not None and time.time() > deadline):
            for i in pending:
                procs[i].kill()
            for i in pending:
                procs[i].wait()
            return rc if rc != 0 else 124
        time.sleep(0.05)
    return rc
