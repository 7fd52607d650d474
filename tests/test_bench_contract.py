"""The one JSON line bench.py prints: keys and types the driver reads.

The reference arm (the fp64 oracle on the host cores) runs without a GPU; the GPU arm is
checked on the smallest configuration with a handful of steps.
"""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e"}


def run_bench(*flags):
    env = dict(os.environ, PYTHONPATH=ROOT)
    for key in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        env.pop(key, None)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                         env=env, cwd=ROOT, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line():
    line = run_bench("--impl", "reference", "--config", "tiny", "--steps", "4", "--warmup", "3")
    assert BASE_KEYS <= set(line)
    assert line["impl"] == "reference" and line["metric"] == "retopk_us_per_decode_step_per_layer"
    assert line["unit"] == "us" and line["higher_is_better"] is False and line["steps"] == 4 and line["warmup"] == 3
    assert line["value"] > 0 and line["dtype"] == "f64" and line["config"]["workload"] == "tiny"
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and cb["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_gpu_arm_line():
    line = run_bench("--config", "tiny", "--steps", "12", "--warmup", "4", "--layers", "2")
    assert BASE_KEYS <= set(line) and "impl" not in line
    assert line["metric"] == "retopk_us_per_decode_step_per_layer" and line["unit"] == "us"
    assert line["n_gpus"] == 1 and line["steps"] == 12 and line["warmup"] == 4 and line["higher_is_better"] is False
    assert line["scaling"] == "weak" and line["vs_baseline"] is None and line["data"] == "synthetic"
    assert line["value"] > 0 and abs(line["ms_per_step"] * 1e3 - line["value"]) < 1e-2
    assert line["gpu_launches"] == 3 * 12
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    roof = line["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-3
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(line["clocks"])
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1


@pytest.mark.gpu
def test_gpu_arm_reports_the_steady_state_and_every_path():
    """Caches are filled before the warm-up, and the step-level and per-path fractions are in the line."""
    line = run_bench("--config", "tiny", "--steps", "12", "--warmup", "4", "--layers", "2", "--no-cpu-baseline")
    cfg = line["config"]
    assert cfg["preroll_steps_per_layer"] >= 16 and cfg["cache_fill_at_first_timed_call"] == 16      # tiny: M = 16
    assert cfg["cache_fill_at_last_timed_call"] == 16
    roof = line["roofline"]
    assert {"recall", "scan", "finish"} <= set(roof["kernels"]) and roof["step"]["frac"] > 0
    for name in ("configured_tau", "pure_reuse", "pure_exact", "tau_0.85"):
        assert line["paths"][name]["us_per_step"] > 0 and roof["paths"][name]["frac"] > 0
    assert abs(line["paths"]["configured_tau"]["us_per_step"] - line["value"]) < 0.02
    assert "met_at_configured_tau" in line["targets"]
    assert line["prefill_seed"]["n_tail"] == 16 and line["prefill_seed"]["ms"] > 0


@pytest.mark.gpu
def test_profiler_case_and_phase_table_run():
    """The small case profiler captures use, and the per-phase clock table of an instrumented
    build (compiled into a temporary directory by the benchmark itself)."""
    env = dict(os.environ, PYTHONPATH=ROOT)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--config", "tiny", "--one-layer", "mix",
                          "--steps", "4", "--preroll", "4"], capture_output=True, text=True, env=env, cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    rec = json.loads([ln for ln in res.stdout.splitlines() if ln.startswith("{")][-1])
    assert rec["one_layer"] == "mix" and rec["steps"] == 8 and rec["stats"]["status"] == 0
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--config", "tiny", "--phases", "--steps", "6",
                          "--preroll", "6"], capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    table = json.loads(res.stdout[res.stdout.index("{"):])
    assert table["pure_reuse"]["recall kernel"]["total"] > 0
    assert table["pure_reuse"]["finish kernel, reuse path"]["total"] > 0
    assert table["pure_exact"]["finish kernel, exact path"]["total"] > 0
