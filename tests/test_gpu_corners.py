"""Parameter corners of the library limits against the oracle (run with -m gpu).

Largest K, largest cache, widest GQA group, both head dims, odd sizes that do not divide
tiles, tiny and long windows: a few teacher-forced steps each, plus Exact Top-K.
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


CASES = [
    # B, H_q, H_kv, d,  context, K,    M,    r, W,    tau,  R, steps
    (1, 16, 1, 64, 9000, 4096, 4, 2, 64, 0.5, 3, 6),      # largest K, widest group, d = 64
    (2, 6, 3, 128, 5003, 77, 1024, 8, 0, 0.6, 0, 8),      # largest cache, no window, odd sizes
    (1, 3, 3, 64, 1234, 512, 5, 5, 3000, 0.7, 2, 7),      # window longer than the history
    (3, 2, 1, 128, 40000, 1000, 9, 3, 17, 0.8, 5, 6),     # several sequences, K not a power of two
    (1, 8, 8, 128, 70000, 2048, 3, 3, 1, 0.3, 0, 5),      # K = 2048 with enough tiles for the bound
    (1, 2, 1, 128, 1048570, 512, 4, 2, 64, 0.4, 0, 4),    # the longest supported history (1 Mi keys)
    (1, 4, 2, 64, 300000, 64, 4, 2, 8, 0.4, 3, 4),        # beyond 256 Ki keys, d = 64
]


@pytest.mark.parametrize("B,H_q,H_kv,d,context,K,M,r,W,tau,R,steps", CASES)
def test_corner_configuration(rt, P, oracle_mod, B, H_q, H_kv, d, context, K, M, r, W, tau, R, steps):
    cfg = wl.Config("corner", 9, B, H_q, H_kv, d, context, steps, K, M, r, W, tau, R, 16, 0.1)
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    P.teacher_forced_run(cfg, st, steps, o, g, k, v)
    so, sg = o.stats(), g.stats()
    for key in ("steps", "refresh"):
        assert sg[key] == so[key], key
    assert sg["status"] == 0
    # Exact Top-K on the last step's inputs
    L = st.seq_len(steps - 1)
    ref_out, ref_idx = o.exact_topk(st.q[steps - 1], st.k, st.v, L)
    import torch
    idx = torch.empty((B, H_q, K), dtype=torch.int32, device="cuda")
    out = g.exact_topk_decode(P.to_dev(st.q[steps - 1]), k, v, L, idx_out=idx)
    idx = idx.cpu().numpy()
    G = H_q // H_kv
    for b in range(B):
        for h in range(H_q):
            sel = ref_idx[b, h][ref_idx[b, h] >= 0]
            q64 = wl.bf16_bits_to_f64(st.q[steps - 1, b, h])
            kth = (wl.bf16_bits_to_f64(st.k[b, h // G, sel]) @ q64 / np.sqrt(d)).min()
            P.assert_support_matches(idx[b, h], ref_idx[b, h], st.q[steps - 1, b, h], st.k[b, h // G], kth,
                                     f"exact seq {b} head {h}")
    P.assert_outputs_close(out, ref_out, "exact_topk_decode")


def _random_config(rng, i):
    G = int(rng.choice([1, 2, 3, 4, 8, 16]))
    H_kv = int(rng.choice([1, 2, 3]))
    d = int(rng.choice([64, 128]))
    K = int(rng.choice([1, 2, 7, 31, 64, 100, 257, 600]))
    M = int(rng.integers(1, 20))
    r = int(rng.integers(1, min(M, 6) + 1))
    W = int(rng.choice([0, 1, 5, 33, 200]))
    context = int(rng.choice([1, 3, 15, 16, 17, 255, 256, 257, 1000, 4100, 9000]))
    return wl.CONFIGS["tiny"].replace(
        name=f"fuzz{i}", B=int(rng.choice([1, 2, 3])), H_q=G * H_kv, H_kv=H_kv, d=d, K=K, M=M, r=r, W=W,
        context=context, steps=int(rng.integers(6, 22)), tau=float(rng.choice([0.3, 0.7, 0.85, 0.95])),
        R=int(rng.choice([0, 1, 3, 8])), n_clusters=4, p_jump=0.1)


@pytest.mark.parametrize("seed", range(40))
def test_random_small_configurations_teacher_forced(rt, P, oracle_mod, seed):
    """Seeded random shapes and hyper-parameters (odd group sizes, K = 1, W = 0, histories shorter
    than K or than one tile, refresh every step ...), every launch shape the library would pick."""
    rng = np.random.default_rng(20260727 + seed)
    cfg = _random_config(rng, seed)
    st = wl.make_stream(cfg, steps=cfg.steps)
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    if seed % 4 == 1:
        g.set_cluster_size(1)
    if seed % 4 == 2:
        g.set_cluster_size(2)
        assert rt.load().retopk_set_finish_threads(g.h, 512) in (0, -2)     # -2: K too large for the narrow shape
    if seed % 4 == 3:
        o.set_qbar_format(1)
        g.set_qbar_format(1)
    P.teacher_forced_run(cfg, st, cfg.steps, o, g, P.to_dev(st.k), P.to_dev(st.v))
    so, sg = o.stats(), g.stats()
    for key in ("steps", "reuse", "fallback", "refresh"):
        assert abs(sg[key] - so[key]) <= 2, (cfg, key, sg, so)       # an excused flip at the tau band at most
    assert sg["status"] == 0


def test_non_finite_inputs_stay_in_bounds(rt, P):
    """NaN and infinities in q / K / V: results are unspecified, but every index the library
    reports lies inside the history, the status word stays clear and the calls return."""
    cfg = wl.CONFIGS["tiny"].replace(context=3000, steps=12, B=2, H_q=4, H_kv=2, d=128, K=100, M=6, r=3, W=20, R=5)
    st = wl.make_stream(cfg, steps=cfg.steps)
    rng = np.random.default_rng(5)
    k, v, q = st.k.copy(), st.v.copy(), st.q.copy()
    specials = np.array([0x7FC0, 0xFFC0, 0x7F80, 0xFF80], dtype=np.uint16)      # +-NaN, +-inf as bf16 bits
    for arr, count in ((k, 4000), (v, 4000), (q, 300)):
        flat = arr.reshape(-1)
        flat[rng.integers(0, flat.size, count)] = specials[rng.integers(0, 4, count)]
    q[3] = 0x7FC0                                                            # one step with an all-NaN query
    g = rt.ReTopK.from_config(cfg)
    kd, vd = P.to_dev(k), P.to_dev(v)
    for t in range(cfg.steps):
        L = st.seq_len(t)
        g.decode_step(P.to_dev(q[t]), kd, vd, L)
        sup = g.last_step()["support"].cpu().numpy()
        assert ((sup >= -1) & (sup < L)).all()
        for row in sup.reshape(-1, cfg.K):
            live = row[row >= 0]
            assert (np.diff(live) > 0).all()                                 # ascending, no duplicates
    assert g.stats()["status"] == 0 and g.stats()["steps"] == cfg.steps * cfg.B * cfg.H_q
