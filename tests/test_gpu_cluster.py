"""Launch shapes of the finish kernel (run with -m gpu).

Thread-block cluster per head: with 2, 4 or 8 CTAs per head the candidate scores and the value
rows are shared out over the CTAs.  Narrow blocks: 512 threads, two CTAs per SM.  Decisions,
supports and candidate counts must not depend on either; outputs may differ in the order of the
fp32 partial sums only.
"""
import pytest
import torch

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


CASES = {
    "d64": wl.CONFIGS["tiny"].replace(context=900, steps=36, B=2, H_q=4, H_kv=2),
    "d128_gqa4": wl.CONFIGS["tiny"].replace(context=5000, steps=36, B=1, H_q=8, H_kv=2, d=128, K=128, M=8, r=3, W=50),
    # fewer selected rows than CTAs: some CTAs get an empty share
    "k3": wl.CONFIGS["tiny"].replace(context=400, steps=24, B=1, H_q=2, H_kv=1, K=3, W=2, r=2, M=4),
    # candidate and support counts that do not divide by the cluster size
    "ragged": wl.CONFIGS["tiny"].replace(context=1000, steps=30, B=1, H_q=3, H_kv=1, K=101, W=7, r=3, M=5),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_cluster_sizes_agree(rt, P, case):
    cfg = CASES[case]
    st = wl.make_stream(cfg, steps=cfg.steps)
    k, v = P.to_dev(st.k), P.to_dev(st.v)

    def run(size, threads=1024):
        g = rt.ReTopK.from_config(cfg)
        g.set_cluster_size(size)
        g.set_finish_threads(threads)
        rec = []
        for t in range(cfg.steps):
            out = g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t))
            ls = g.last_step()
            idx = torch.empty((cfg.B, cfg.H_q, cfg.K), dtype=torch.int32, device="cuda")
            ex = g.exact_topk_decode(P.to_dev(st.q[t]), k, v, st.seq_len(t), idx_out=idx)
            rec.append((out.float().clone(), ls["support"].clone(), ls["path"].clone(), ls["rho_max"].clone(),
                        ls["n_cand"].clone(), ex.float().clone(), idx))
        return rec, g.stats()

    ref, ref_stats = run(1)
    assert ref_stats["reuse"] > 0 and ref_stats["fallback"] + ref_stats["refresh"] > 0
    for size, threads in ((2, 1024), (4, 1024), (8, 1024), (1, 512), (2, 512)):
        rec, stats = run(size, threads)
        assert stats == ref_stats, (size, stats, ref_stats)
        for t, (a, b) in enumerate(zip(ref, rec)):
            for name, x, y in zip(("out", "support", "path", "rho_max", "n_cand", "exact_out", "exact_idx"), a, b):
                if name in ("out", "exact_out"):
                    # bf16 outputs of fp32 sums taken in another order: one bf16 step at most
                    assert torch.allclose(x, y, rtol=2 ** -7, atol=1e-6), (size, t, name)
                else:
                    assert torch.equal(x, y), (size, t, name)


def test_shapes_against_the_oracle(rt, P, oracle_mod):
    cfg = wl.CONFIGS["tiny"].replace(context=2500, steps=24, B=1, H_q=8, H_kv=2, d=128, K=96, M=8, r=3, W=40)
    st = wl.make_stream(cfg, steps=cfg.steps)
    for size, threads in ((4, 1024), (8, 1024), (1, 512)):
        o = oracle_mod.Oracle.from_config(cfg)
        g = rt.ReTopK.from_config(cfg)
        g.set_cluster_size(size)
        g.set_finish_threads(threads)
        P.teacher_forced_run(cfg, st, cfg.steps, o, g, P.to_dev(st.k), P.to_dev(st.v))
        so, sg = o.stats(), g.stats()
        assert so["reuse"] > 0
        for key in ("steps", "reuse", "fallback", "refresh", "cand_sum"):
            assert sg[key] == so[key], (size, key)


def test_cluster_argument_checks(rt):
    g = rt.ReTopK.from_config(wl.CONFIGS["tiny"])
    lib = rt.load()
    for bad in (0, 3, 16, -1):
        assert lib.retopk_set_cluster_size(g.h, bad) == -1
    assert lib.retopk_set_cluster_size(None, 2) == -1
    for ok in (1, 2, 4, 8):
        assert lib.retopk_set_cluster_size(g.h, ok) == 0
    for bad in (0, 256, 768, 2048):
        assert lib.retopk_set_finish_threads(g.h, bad) == -1
    assert lib.retopk_set_finish_threads(g.h, 512) == 0 and lib.retopk_set_finish_threads(g.h, 1024) == 0
    # a support size whose lists do not fit half an SM's shared memory
    big = rt.ReTopK.from_config(wl.CONFIGS["tiny"].replace(K=2048, r=8, W=512, context=20000, steps=4))
    assert lib.retopk_set_finish_threads(big.h, 512) == -2
