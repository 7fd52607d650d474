"""The allocation-free Exact Top-K entry point against the context-based one and against the
fp64 oracle (run with -m gpu).

Some callers cannot call cudaMalloc: their device memory belongs to another allocator, or
they are plug-ins that only receive input and output buffers.  For them the library keeps the
score workspace in a fixed array inside the library image.  This file is collected last so
that a failure here cannot hide the other tests' results in a stop-at-first-failure run; it
passes both on its own in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from paper_2607_27692_b200 import workload as wl

pytestmark = pytest.mark.gpu


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


@pytest.mark.parametrize("B,H_q,H_kv,d,K,Lmax,lengths", [
    (2, 8, 2, 128, 256, 20000, (19990, 7001)),      # 16 heads: a cluster of CTAs per head
    (1, 4, 1, 64, 100, 9000, (8999, 515)),          # head dim 64
    (5, 16, 4, 128, 64, 3000, (2999, 1300)),        # 80 heads: one CTA per head
])
def test_static_entry_point_matches_context_entry_point_and_oracle(oracle_mod, B, H_q, H_kv, d, K, Lmax, lengths):
    from paper_2607_27692_b200 import build, retopk as rt
    build.build()
    rng = np.random.default_rng(77 + d + B)
    k_bits = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    v_bits = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    k = rt.bf16_tensor_from_bits(k_bits, device="cuda")
    v = rt.bf16_tensor_from_bits(v_bits, device="cuda")
    ctx = rt.ReTopK(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, Lmax)
    ref = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, Lmax)
    # outputs are allocated once, up front, as a caller that may not allocate later would do
    out_s = torch.empty((B, H_q, d), dtype=torch.bfloat16, device="cuda")
    idx_s = torch.empty((B, H_q, K), dtype=torch.int32, device="cuda")
    out_c = torch.empty_like(out_s)
    idx_c = torch.empty_like(idx_s)
    # two calls in a row on different inputs and lengths: the second must not see the first's scratch
    for call, L in enumerate(lengths):
        q_bits = bits(rng.standard_normal((B, H_q, d)))
        q = rt.bf16_tensor_from_bits(q_bits, device="cuda")
        out_s.zero_()
        idx_s.fill_(-5)
        rt.exact_topk_decode_static(q, k, v, L, K, out=out_s, idx_out=idx_s)
        ctx.exact_topk_decode(q, k, v, L, out=out_c, idx_out=idx_c)
        torch.cuda.synchronize()
        assert torch.equal(idx_s, idx_c), f"call {call}: supports differ"
        got, want = out_s.float().cpu().numpy(), out_c.float().cpu().numpy()
        assert (np.abs(got - want) <= 2e-2 + 1e-2 * np.abs(want)).all(), f"call {call}"
        assert torch.equal(out_s.view(torch.int16), out_c.view(torch.int16)), f"call {call}: same kernels, same bits"
        # and against the fp64 oracle, under the library's parity rules
        o_out, o_idx = ref.exact_topk(q_bits, k_bits, v_bits, L)
        G = H_q // H_kv
        got_idx = idx_s.cpu().numpy()
        import math
        for b in range(B):
            for h in range(H_q):
                a, w = got_idx[b, h], o_idx[b, h]
                diff = np.setxor1d(a[a >= 0], w[w >= 0])
                if len(diff):
                    q64 = wl.bf16_bits_to_f64(q_bits[b, h])
                    sc = wl.bf16_bits_to_f64(k_bits[b, h // G]) @ q64 / math.sqrt(d)
                    kth = np.sort(sc[:L])[-min(K, L)]
                    assert (np.abs(sc[diff] - kth) <= 1e-3 * abs(kth)).all(), f"call {call} head {b},{h}"
        assert (np.abs(got - o_out) <= 2e-2 + 1e-2 * np.abs(o_out)).all(), f"call {call}: against the oracle"


def test_static_entry_point_rejects_shapes_beyond_its_array():
    from paper_2607_27692_b200 import build, retopk as rt
    build.build()
    lib = rt.load()
    # 128 heads x 131584 keys needs about 72 MB of scores: more than the fixed 32 MiB
    one = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    p = one.data_ptr()
    rc = lib.exact_topk_decode_static(4, 32, 8, 128, 512, 131584, p, p, p, 1000, p, None, None)
    assert rc == -5
    assert b"fixed scratch" in lib.retopk_strerror(rc)
    with pytest.raises(rt.RetopkError):
        big = torch.zeros((1, 64, 131072, 128), dtype=torch.bfloat16, device="cuda")
        rt.exact_topk_decode_static(torch.zeros((1, 64, 128), dtype=torch.bfloat16, device="cuda"), big, big, 10, 64)
