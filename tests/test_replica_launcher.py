"""bench.py --gpus N starts its own replicas: the launcher driven on CPU with a stub worker.

Two gloo ranks are spawned exactly as the benchmark spawns its GPU replicas (same function,
same environment variables); each joins the process group, takes part in the barrier and the
max-over-ranks reduction the benchmark uses for its timing, and rank 0 prints the line.
"""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import json, os, sys
sys.path.insert(0, {root!r})
from paper_2607_27692_b200 import replicas
rank, world, local = replicas.rank_info()
assert replicas.under_launcher() and local == rank
dist = replicas.init("gloo")
replicas.barrier(dist)
slowest = replicas.max_over_ranks(10.0 * (rank + 1), dist)
if len(sys.argv) > 1 and sys.argv[1] == "fail" and rank == 1:
    sys.exit(7)
replicas.barrier(dist)
if rank == 0:
    print(json.dumps({{"n_gpus": world, "slowest": slowest, "cost": replicas.job_cost_per_step(slowest, world)}}), flush=True)
else:
    print("noise from rank", rank, flush=True)      # must not reach the job's stdout
dist.destroy_process_group()
'''


def _run(tmp_path, *extra):
    worker = tmp_path / "worker.py"
    worker.write_text(WORKER.format(root=ROOT))
    driver = (f"import sys; sys.path.insert(0, {ROOT!r}); from paper_2607_27692_b200 import replicas; "
              f"sys.exit(replicas.spawn([sys.executable, {str(worker)!r}] + sys.argv[1:], 2, timeout=120))")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    return subprocess.run([sys.executable, "-c", driver, *extra], capture_output=True, text=True, timeout=180, env=env)


def test_two_replicas_are_spawned_and_rank_zero_prints_the_line(tmp_path):
    res = _run(tmp_path)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line == {"n_gpus": 2, "slowest": 20.0, "cost": 10.0}


def test_a_failing_rank_ends_the_job_with_its_code(tmp_path):
    res = _run(tmp_path, "fail")
    assert res.returncode == 7


def test_bench_spawns_only_without_a_launcher(monkeypatch):
    from paper_2607_27692_b200 import replicas
    monkeypatch.delenv("RANK", raising=False)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    assert not replicas.under_launcher()
    monkeypatch.setenv("RANK", "0")
    monkeypatch.setenv("WORLD_SIZE", "2")
    assert replicas.under_launcher()
