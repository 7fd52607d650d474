"""The allocation-free Exact Top-K entry point against the context-based one (run with -m gpu).

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


def test_static_entry_point_matches_context_entry_point():
    from paper_2607_27692_b200 import build, retopk as rt
    build.build()
    B, H_q, H_kv, d, K, Lmax = 2, 8, 2, 128, 256, 20000
    rng = np.random.default_rng(77)
    k = rt.bf16_tensor_from_bits(bits(rng.standard_normal((B, H_kv, Lmax, d))), device="cuda")
    v = rt.bf16_tensor_from_bits(bits(rng.standard_normal((B, H_kv, Lmax, d))), device="cuda")
    ctx = rt.ReTopK(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, Lmax)
    # outputs are allocated once, up front, as a caller that may not allocate later would do
    out_s = torch.empty((B, H_q, d), dtype=torch.bfloat16, device="cuda")
    idx_s = torch.empty((B, H_q, K), dtype=torch.int32, device="cuda")
    out_c = torch.empty_like(out_s)
    idx_c = torch.empty_like(idx_s)
    # two calls in a row on different inputs and lengths: the second must not see the first's scratch
    for call, L in enumerate((19990, 7001)):
        q = rt.bf16_tensor_from_bits(bits(rng.standard_normal((B, H_q, d))), device="cuda")
        out_s.zero_()
        idx_s.fill_(-5)
        rt.exact_topk_decode_static(q, k, v, L, K, out=out_s, idx_out=idx_s)
        ctx.exact_topk_decode(q, k, v, L, out=out_c, idx_out=idx_c)
        torch.cuda.synchronize()
        assert torch.equal(idx_s, idx_c), f"call {call}: supports differ"
        got, want = out_s.float().cpu().numpy(), out_c.float().cpu().numpy()
        assert (np.abs(got - want) <= 2e-2 + 1e-2 * np.abs(want)).all(), f"call {call}"
        assert torch.equal(out_s.view(torch.int16), out_c.view(torch.int16)), f"call {call}: same kernels, same bits"


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
