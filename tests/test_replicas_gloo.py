"""Two CPU ranks over gloo: the barrier / max-over-ranks plumbing of multi-GPU benchmark runs."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2607_27692_b200 import replicas
    assert replicas.rank_info() == (rank, world, rank)
    dist = replicas.init("gloo")
    assert dist is not None and dist.get_world_size() == world
    replicas.barrier(dist)
    slowest = replicas.max_over_ranks(10.0 + 5.0 * rank, dist)     # rank 1 is the slow replica
    out.put((rank, slowest, replicas.job_cost_per_step(slowest, world)))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 7.5), (1, 15.0, 7.5)]


def test_single_process_needs_no_group(monkeypatch):
    for key in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        monkeypatch.delenv(key, raising=False)
    from paper_2607_27692_b200 import replicas
    assert replicas.rank_info() == (0, 1, 0)
    assert replicas.init("gloo") is None
    assert replicas.max_over_ranks(3.5, None) == 3.5
    assert replicas.job_cost_per_step(8.0, 1) == 8.0
