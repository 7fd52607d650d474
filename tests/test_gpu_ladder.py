"""Fusion ladder (run with -m gpu): every level of the reuse path gives the production result.

Levels 1-4 run the reuse path as separate kernels with their intermediates in global memory
(Table 4 of the paper reports such a ladder).  They execute the same device functions on the
same lanes, so free-running runs with one CTA per head must agree with the default level bit for bit: outputs,
supports, paths, candidate counts, similarity maxima and the path counters.  One level is
also checked against the fp64 oracle directly.
"""
import pytest
import torch

from paper_2607_27692_b200 import workload as wl

pytestmark = pytest.mark.gpu

LEVELS = [(1, False), (2, False), (3, False), (4, False), (5, False)]


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


CASES = {
    "tiny_d64": (wl.CONFIGS["tiny"].replace(context=900, steps=40, B=2, H_q=4, H_kv=2), {}),
    "d128_gqa4": (wl.CONFIGS["tiny"].replace(context=5000, steps=40, B=2, H_q=8, H_kv=2, d=128, K=128, M=8, r=3, W=50),
                  {}),
    "recent_recall": (wl.CONFIGS["tiny"].replace(context=700, steps=30, B=1, H_q=4, H_kv=1, M=6, r=3), {"recent": True}),
    "few_candidates": (wl.CONFIGS["tiny"].replace(context=300, steps=24, B=1, H_q=2, H_kv=1, K=200, W=0, r=1), {}),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_levels_agree_bit_for_bit(rt, P, case):
    cfg, opt = CASES[case]
    st = wl.make_stream(cfg, steps=cfg.steps)
    k, v = P.to_dev(st.k), P.to_dev(st.v)

    def run(level):
        g = rt.ReTopK.from_config(cfg)
        g.set_cluster_size(1)          # the unfused kernels run one CTA per head
        if opt.get("recent"):
            g.set_recall_mode(1)
        if level is not None:
            g.set_fusion_level(*level)
        rec = []
        for t in range(cfg.steps):
            out = g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t))
            ls = g.last_step()
            rec.append((out.view(torch.int16).clone(), ls["support"].clone(), ls["path"].clone(),
                        ls["rho_max"].clone(), ls["n_cand"].clone()))
        return rec, g.stats(), g.last_launch_count()

    ref, ref_stats, ref_launches = run(None)
    assert ref_launches == 3
    assert ref_stats["reuse"] > 0 and ref_stats["fallback"] + ref_stats["refresh"] > 0
    expected_launches = {1: 10, 2: 7, 3: 5, 4: 5, 5: 3}
    for level in LEVELS:
        rec, stats, launches = run(level)
        assert launches == expected_launches[level[0]], (level, launches)
        assert stats == ref_stats, (level, stats, ref_stats)
        for t, (a, b) in enumerate(zip(ref, rec)):
            for name, x, y in zip(("out", "support", "path", "rho_max", "n_cand"), a, b):
                assert torch.equal(x, y), (level, t, name)


def test_level_one_against_the_oracle(rt, P, oracle_mod):
    cfg = wl.CONFIGS["tiny"].replace(context=2000, steps=24, B=2, H_q=8, H_kv=2, d=128, K=96, M=8, r=3, W=40)
    st = wl.make_stream(cfg, steps=cfg.steps)
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    g.set_fusion_level(1)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    P.teacher_forced_run(cfg, st, cfg.steps, o, g, k, v)
    so, sg = o.stats(), g.stats()
    assert so["reuse"] > 0 and sg["steps"] == so["steps"] and sg["status"] == 0


def test_level_arguments(rt):
    cfg = wl.CONFIGS["tiny"]
    g = rt.ReTopK.from_config(cfg)
    lib = rt.load()
    assert lib.retopk_set_fusion_level(g.h, 0, 0) == -1
    assert lib.retopk_set_fusion_level(g.h, 6, 0) == -1
    assert lib.retopk_set_fusion_level(g.h, 3, 1) == -1      # dependent launches only at level 5
    assert lib.retopk_set_fusion_level(g.h, 5, 2) == -1
    assert lib.retopk_set_fusion_level(None, 5, 1) == -1
    assert lib.retopk_set_fusion_level(g.h, 2, 0) == 0
    assert lib.retopk_set_fusion_level(g.h, 5, 1) == 0
