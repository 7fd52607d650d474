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
