"""Recall, candidate union and ring wrap with caches that are FULL from the first step (run
with -m gpu).  The benchmark's steady state has every cache full (fill = M), a launch shape the
stream tests only reach after M steps; here the same synthetic full state is written into the
fp64 oracle and imported into the GPU context, then both step teacher-forced for at least M/4
steps so that the ring's write position wraps or overwrites recalled entries.

Cache sizes cover every thread split of the Top-r ranking (entries per thread group) and the
second trip of the similarity loop (more than 128 entries at 1024 threads); r in {1, 4, 8};
both storage formats of the cached queries; recency recall; exact similarity ties between slots.
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


def run_full(rt, P, oracle_mod, cfg, steps, seed, bf16=False, recent=False, n_inserted=None, dup_slots=(), **override):
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg, **override)
    g = rt.ReTopK.from_config(cfg, **override)
    if bf16:
        o.set_qbar_format(1)
        g.set_qbar_format(1)
        o.qbar_bf16 = True
    if recent:
        o.set_recall_mode(1)
        g.set_recall_mode(1)
    P.synthetic_full_state(o, st, cfg.context, np.random.default_rng(seed), n_inserted=n_inserted, dup_slots=dup_slots)
    ex = P.teacher_forced_run(cfg, st, steps, o, g, P.to_dev(st.k), P.to_dev(st.v))
    so, sg = o.stats(), g.stats()
    assert abs(sg["reuse"] - so["reuse"]) <= ex["flips"]
    assert sg["status"] == 0
    return so, sg, ex, o, g


@pytest.mark.parametrize("M,r,d", [(64, 4, 128), (128, 4, 128), (128, 8, 64), (300, 1, 128), (300, 8, 128),
                                   (1024, 4, 128), (1024, 8, 64), (17, 4, 128), (33, 8, 64)])
def test_full_cache_teacher_forced(rt, P, oracle_mod, M, r, d):
    """Top-r over a full cache of M entries; the ring wraps during the run."""
    steps = max(12, M // 4)
    cfg = wl.CONFIGS["tiny"].replace(B=1, H_q=4, H_kv=2, d=d, context=3000, steps=steps, K=96, W=40, M=M, r=r,
                                     tau=0.55, R=0)
    so, sg, ex, o, g = run_full(rt, P, oracle_mod, cfg, steps, seed=1000 + M + r, n_inserted=2 * M - steps // 2)
    assert so["reuse"] > 0, "the synthetic cache must let some heads reuse"
    # the ring position passed M again: the write slot wrapped during the run
    assert o.export_state()[2] == 2 * M - steps // 2 + steps


@pytest.mark.parametrize("M", [128, 1024])
def test_full_cache_with_bf16_queries(rt, P, oracle_mod, M):
    steps = M // 4
    cfg = wl.CONFIGS["tiny"].replace(B=1, H_q=4, H_kv=2, d=128, context=2500, steps=steps, K=64, W=24, M=M, r=4,
                                     tau=0.55, R=0)
    so, *_ = run_full(rt, P, oracle_mod, cfg, steps, seed=7 + M, bf16=True)
    assert so["reuse"] > 0


@pytest.mark.parametrize("M,r", [(128, 4), (300, 8)])
def test_full_cache_with_recency_recall(rt, P, oracle_mod, M, r):
    steps = M // 4
    cfg = wl.CONFIGS["tiny"].replace(B=1, H_q=4, H_kv=2, d=128, context=2500, steps=steps, K=64, W=24, M=M, r=r,
                                     tau=0.3, R=0)
    so, *_ = run_full(rt, P, oracle_mod, cfg, steps, seed=70 + M, recent=True)
    assert so["reuse"] > 0


def test_exact_similarity_ties_between_slots(rt, P, oracle_mod):
    """Identical cached queries in different slots tie exactly: the lower slot is recalled first
    on both sides (compared through the candidate lists and supports, and through last_recall)."""
    M, r, steps = 128, 4, 16
    cfg = wl.CONFIGS["tiny"].replace(B=1, H_q=4, H_kv=2, d=128, context=2500, steps=steps, K=64, W=24, M=M, r=r,
                                     tau=-2.0, R=0)
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    # slots 0..5 hold near copies of the query direction; (0,3), (1,100), (2,127) are exact duplicates
    P.synthetic_full_state(o, st, cfg.context, np.random.default_rng(5), n_inserted=M + 40,
                           dup_slots=((0, 3), (1, 100), (2, 127)))
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    import torch
    for t in range(steps):
        qbar, sup, n_ins, t_dec = o.export_state()
        g.import_state(torch.from_numpy(qbar.astype(np.float32)).cuda(), torch.from_numpy(sup).cuda(), n_ins, t_dec)
        g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t))
        o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        sel_o = o.last_step()["sel"]
        sel_g = g.last_recall().cpu().numpy()
        qn = qbar.astype(np.float32).astype(np.float64)
        for h in range(cfg.H_q):
            if not np.array_equal(sel_g[0, h], sel_o[0, h]):
                # only near-ties in fp32 vs fp64 may differ; exact duplicates never
                rho = qn[0, h] @ (wl.bf16_bits_to_f64(st.q[t, 0, h]) / np.linalg.norm(wl.bf16_bits_to_f64(st.q[t, 0, h])))
                a, b = rho[sel_g[0, h]], rho[sel_o[0, h]]
                assert np.allclose(np.sort(a), np.sort(b), atol=2e-6), (t, h, sel_g[0, h], sel_o[0, h])
            for lo, hi in ((0, 3), (1, 100), (2, 127)):
                s = list(sel_g[0, h])
                if hi in s:
                    assert lo in s and s.index(lo) < s.index(hi), f"step {t} head {h}: tie not resolved to the lower slot: {s}"


def test_headline_shape_from_a_full_cache(rt, P, oracle_mod):
    """The benchmark's launch shape in its steady state: 128K context, batch 4, M = 128 full,
    candidate sets near the capacity r*K + W (random supports barely overlap)."""
    cfg = wl.CONFIGS["headline128k"]
    steps, sample = 6, [2]
    full = wl.make_stream(cfg, steps=steps)
    sub = wl.Stream(cfg.replace(B=1), np.ascontiguousarray(full.k[sample]), np.ascontiguousarray(full.v[sample]),
                    np.ascontiguousarray(full.q[:, sample]))
    o = oracle_mod.Oracle.from_config(sub.cfg, tau=0.6, R=0)
    g = rt.ReTopK.from_config(cfg, tau=0.6, R=0)
    P.synthetic_full_state(o, sub, cfg.context, np.random.default_rng(99), n_inserted=cfg.M + 125)
    # the other sequences of the batch start from the same kind of state
    import torch
    qbar, sup, n_ins, t_dec = o.export_state()
    g.import_state(torch.from_numpy(np.repeat(qbar, cfg.B, 0).astype(np.float32)).cuda(),
                   torch.from_numpy(np.repeat(sup, cfg.B, 0)).cuda(), n_ins, t_dec)
    ex = P.teacher_forced_run(cfg, sub, steps, o, g, P.to_dev(full.k), P.to_dev(full.v), b_map=sample, full_stream=full)
    so, sg = o.stats(), g.stats()
    assert so["reuse"] > 0 and so["cand_sum"] / so["reuse"] > 1500
    assert sg["status"] == 0 and sg["slow_select"] == 0


@pytest.mark.parametrize("threads,per_sm", [(512, 1), (512, 2)])
@pytest.mark.parametrize("d", [64, 128])
def test_block_shapes_against_the_oracle(rt, P, oracle_mod, threads, per_sm, d):
    """Every block shape of the per-head kernels, full cache, both paths (tau in the middle of the similarities)."""
    M, r, steps = 128, 4, 24
    cfg = wl.CONFIGS["tiny"].replace(B=2, H_q=4, H_kv=2, d=d, context=5000, steps=steps, K=128, W=48, M=M, r=r,
                                     tau=0.9, R=8)
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    g.set_block_shape(threads, per_sm)
    P.synthetic_full_state(o, st, cfg.context, np.random.default_rng(threads + d), n_inserted=M + 100)
    ex = P.teacher_forced_run(cfg, st, steps, o, g, P.to_dev(st.k), P.to_dev(st.v))
    so, sg = o.stats(), g.stats()
    assert so["reuse"] > 0 and so["fallback"] + so["refresh"] > 0
    assert abs(sg["reuse"] - so["reuse"]) <= ex["flips"] and sg["status"] == 0
