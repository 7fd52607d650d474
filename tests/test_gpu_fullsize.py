"""Full-size parity (run with -m gpu): the configurations the benchmark times, at their real
batch, context and launch shapes.  The GPU runs the whole batch; the fp64 oracle follows
sampled sequences (sequences are independent, so a sampled sequence is generated and checked
on its own) with the GPU caches re-seeded from it before every step.
"""
import numpy as np
import pytest

from paper_2607_27692_b200 import workload as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rt():
    from paper_2607_27692_b200 import build, retopk
    build.build()
    retopk.load()
    return retopk


@pytest.fixture(scope="module")
def P():
    import parity
    return parity


def run_sampled(rt, P, oracle_mod, name, steps, sample, **override):
    cfg = wl.CONFIGS[name]
    full = wl.make_stream(cfg, steps=steps)
    sub = wl.Stream(cfg.replace(B=len(sample)), np.ascontiguousarray(full.k[sample]),
                    np.ascontiguousarray(full.v[sample]), np.ascontiguousarray(full.q[:, sample]))
    # a sampled sequence generated on its own is the same data
    alone = wl.make_stream(cfg, steps=steps, sequences=range(sample[0], sample[0] + 1))
    assert np.array_equal(alone.k[0], sub.k[0]) and np.array_equal(alone.q[:, 0], sub.q[:, 0])
    o = oracle_mod.Oracle.from_config(sub.cfg, **override)
    g = rt.ReTopK.from_config(cfg, **override)
    k, v = P.to_dev(full.k), P.to_dev(full.v)
    ex = P.teacher_forced_run(cfg, sub, steps, o, g, k, v, b_map=list(sample), full_stream=full)
    return o.stats(), g.stats(), ex


@pytest.mark.parametrize("name", ["batch32k", "batch64k"])
def test_batched_configs(rt, P, oracle_mod, name):
    so, sg, ex = run_sampled(rt, P, oracle_mod, name, 12, [0, 5])
    assert so["reuse"] > 0 and so["fallback"] > 0
    assert sg["steps"] == 12 * 8 * 32 and sg["slow_select"] == 0 and sg["status"] == 0


def test_headline_config(rt, P, oracle_mod):
    """128K context, batch 4, K = 512, M = 128, r = 4, W = 256; 34 steps reach the first refresh."""
    so, sg, ex = run_sampled(rt, P, oracle_mod, "headline128k", 34, [1, 3])
    assert so["refresh"] == 2 * 32 and so["reuse"] > 0 and so["fallback"] > 0
    assert sg["steps"] == 34 * 4 * 32 and sg["slow_select"] == 0 and sg["status"] == 0


def test_headline_shapes_with_k1024(rt, P, oracle_mod):
    """The cross-model 128K setting (Table 2) keeps K = 1024 keys per head."""
    so, sg, ex = run_sampled(rt, P, oracle_mod, "headline128k_k1024", 10, [2], tau=0.85)
    assert so["reuse"] > 0 and so["fallback"] > 0
    assert sg["steps"] == 10 * 4 * 32 and sg["slow_select"] == 0 and sg["status"] == 0


def test_single_sequence_at_128k(rt, P, oracle_mod):
    """Batch 1 at 128K (the paper's latency setting): four CTAs per head in the finish kernel."""
    so, sg, ex = run_sampled(rt, P, oracle_mod, "single128k", 8, [0], tau=0.85)
    assert so["reuse"] > 0 and so["fallback"] > 0
    assert sg["steps"] == 8 * 32 and sg["slow_select"] == 0 and sg["status"] == 0


def test_stress_config(rt, P, oracle_mod):
    """128K, batch 16, K = 2048, r = 8, W = 512, refresh every 8 steps: mostly exact steps."""
    so, sg, ex = run_sampled(rt, P, oracle_mod, "stress128k", 10, [9])
    assert so["refresh"] == 32 and so["fallback"] > so["reuse"]
    assert sg["steps"] == 10 * 16 * 32 and sg["slow_select"] == 0


def test_stress_shapes_on_the_reuse_path(rt, P, oracle_mod):
    """Same shapes with a low threshold: candidate sets of up to 8*2048 + 512 keys."""
    so, sg, ex = run_sampled(rt, P, oracle_mod, "stress128k", 6, [2], tau=0.3, R=0)
    assert so["reuse"] >= 4 * 32 and so["cand_sum"] / so["reuse"] > 2048
