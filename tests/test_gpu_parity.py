"""GPU parity: the CUDA library against the fp64 oracle, element by element (run with -m gpu).

Rules: path decisions and index sets are bit-exact except for positions whose fp64 score is
within 1e-3 relative of the K-th score and steps whose rho_max is within 1e-4 of tau;
outputs within 2e-2 absolute + 1e-2 relative (bf16 I/O, fp32 accumulation).  In the
teacher-forced runs the GPU caches are overwritten with the oracle's before every step so
that an excused difference cannot compound.
"""
import json
import os

import numpy as np
import pytest
import torch

from paper_2607_27692_b200 import workload as wl

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


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


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ------------------------------------------------------------------ Exact Top-K

@pytest.mark.parametrize("B,H_q,H_kv,d,L,K,Lmax", [
    (1, 1, 1, 64, 2112, 64, 2112),        # the tiny configuration's shape
    (2, 8, 2, 128, 5000, 512, 5003),      # several scan tiles and a ragged tail
    (1, 4, 4, 128, 9000, 100, 9001),      # longer than the threshold sample
    (1, 16, 1, 64, 777, 33, 800),         # two head tiles per group
    (1, 2, 1, 128, 300, 512, 300),        # fewer keys than K
    (1, 32, 8, 128, 20000, 2048, 20480),  # large K, fewer 16-row tiles than K: multi-pass select
    (1, 8, 2, 128, 40000, 2048, 40000),   # large K with enough tiles for the tile-maximum bound
])
def test_exact_topk_decode_matches_oracle(rt, P, oracle_mod, B, H_q, H_kv, d, L, K, Lmax):
    rng = np.random.default_rng(L + K)
    k = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    v = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    q = bits(rng.standard_normal((B, H_q, d)))
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, Lmax)
    ref_out, ref_idx = o.exact_topk(q, k, v, L)
    g = rt.ReTopK(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, Lmax)
    idx = torch.full((B, H_q, K), -7, dtype=torch.int32, device="cuda")
    out = g.exact_topk_decode(P.to_dev(q), P.to_dev(k), P.to_dev(v), L, idx_out=idx)
    idx = idx.cpu().numpy()
    G = H_q // H_kv
    for b in range(B):
        for h in range(H_q):
            srt = np.sort(ref_idx[b, h][ref_idx[b, h] >= 0])
            q64 = wl.bf16_bits_to_f64(q[b, h])
            kth = (wl.bf16_bits_to_f64(k[b, h // G, srt]) @ q64 / np.sqrt(d)).min()
            P.assert_support_matches(idx[b, h], ref_idx[b, h], q[b, h], k[b, h // G], kth,
                                     f"seq {b} head {h}")
    P.assert_outputs_close(out, ref_out, "exact_topk_decode")
    # the tile-maximum bound needs at least K 16-row tiles, or all of L must fit the shared list
    list_capacity = 16384 if K > 512 else 8192
    fast = L <= K or -(-L // 16) >= K or L <= list_capacity
    assert g.stats()["slow_select"] == (0 if fast else B * H_q)
    assert g.last_launch_count() == 2


def test_exact_ties_are_bit_exact(rt, P, oracle_mod):
    """Integer inputs: scores tie exactly and are exact in fp32, so indices must be identical."""
    B, H_q, H_kv, d, L, K = 1, 4, 2, 64, 3000, 128
    rng = np.random.default_rng(11)
    kf = rng.integers(-2, 3, size=(B, H_kv, L, d)).astype(np.float32)
    kf[0, 0, 5] = 0.0
    kf[0, 0, 6] = -0.0
    qf = rng.integers(-1, 2, size=(B, H_q, d)).astype(np.float32)
    k, v, q = bits(kf), bits(rng.standard_normal((B, H_kv, L, d))), bits(qf)
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, L)
    ref_out, ref_idx = o.exact_topk(q, k, v, L)
    g = rt.ReTopK(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, L)
    idx = torch.empty((B, H_q, K), dtype=torch.int32, device="cuda")
    out = g.exact_topk_decode(P.to_dev(q), P.to_dev(k), P.to_dev(v), L, idx_out=idx)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    P.assert_outputs_close(out, ref_out, "ties")


def test_degenerate_scores_take_the_multi_pass_path(rt, P, oracle_mod):
    """All keys identical: every score ties, the support is the first K indices."""
    B, H_q, H_kv, d, L, K = 1, 2, 1, 128, 20000, 512
    rng = np.random.default_rng(12)
    k = np.broadcast_to(bits(rng.standard_normal((1, 1, 1, d))), (B, H_kv, L, d)).copy()
    v = bits(rng.standard_normal((B, H_kv, L, d)))
    q = bits(rng.standard_normal((B, H_q, d)))
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, L)
    ref_out, ref_idx = o.exact_topk(q, k, v, L)
    assert np.array_equal(ref_idx[0, 0], np.arange(K))
    g = rt.ReTopK(B, H_q, H_kv, d, 4, 2, 8, K, 0.9, 0, L)
    idx = torch.empty((B, H_q, K), dtype=torch.int32, device="cuda")
    out = g.exact_topk_decode(P.to_dev(q), P.to_dev(k), P.to_dev(v), L, idx_out=idx)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    P.assert_outputs_close(out, ref_out, "degenerate")
    assert g.stats()["slow_select"] == B * H_q


# ------------------------------------------------------------------ ReTopK steps

def stream_case(rt, P, oracle_mod, cfg, steps, **override):
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg, **override)
    g = rt.ReTopK.from_config(cfg, **override)
    return st, o, g, P.to_dev(st.k), P.to_dev(st.v)


def test_tiny_config_teacher_forced(rt, P, oracle_mod):
    cfg = wl.CONFIGS["tiny"]
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, cfg.steps)
    ex = P.teacher_forced_run(cfg, st, cfg.steps, o, g, k, v)
    so, sg = o.stats(), g.stats()
    assert ex["flips"] == 0
    for key in ("steps", "reuse", "fallback", "refresh", "cand_sum"):
        assert sg[key] == so[key], key
    assert so["reuse"] > so["fallback"] > 0 and so["refresh"] == 3
    assert sg["status"] == 0


@pytest.mark.parametrize("override", [{"r": 1}, {"M": 1, "r": 1}, {"W": 0}, {"R": 0}, {"tau": -2.0},
                                      {"tau": 2.0}, {"K": 300, "W": 5}])
def test_parameter_corners_teacher_forced(rt, P, oracle_mod, override):
    cfg = wl.CONFIGS["tiny"].replace(context=700, steps=24, B=2, H_q=4, H_kv=2)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, 24, **override)
    P.teacher_forced_run(cfg, st, 24, o, g, k, v)
    so, sg = o.stats(), g.stats()
    for key in ("steps", "reuse", "fallback", "refresh", "cand_sum"):
        assert sg[key] == so[key], key


def test_llama_shape_teacher_forced(rt, P, oracle_mod):
    """32 query / 8 KV heads, d = 128, 16K context: the second configuration, first 40 steps."""
    cfg = wl.CONFIGS["llama16k"]
    steps = 40
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, steps)
    ex = P.teacher_forced_run(cfg, st, steps, o, g, k, v)
    so, sg = o.stats(), g.stats()
    assert so["reuse"] > 0 and so["fallback"] > 0 and so["refresh"] == 32
    # counters agree up to the excused decisions
    assert abs(sg["reuse"] - so["reuse"]) <= ex["flips"]
    assert sg["slow_select"] == 0 and sg["status"] == 0


def test_free_running_stays_close(rt, P, oracle_mod):
    """No re-seeding: decisions may drift apart at excused ties, outputs must stay aligned."""
    cfg = wl.CONFIGS["tiny"].replace(B=2, H_q=4, H_kv=2)
    steps = 48
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, steps)
    cos = []
    for t in range(steps):
        L = st.seq_len(t)
        out_g = g.decode_step(P.to_dev(st.q[t]), k, v, L).float().cpu().numpy().astype(np.float64)
        out_o = o.decode_step(st.q[t], st.k, st.v, L)
        cos.append((out_g * out_o).sum(-1) / (np.linalg.norm(out_g, axis=-1) * np.linalg.norm(out_o, axis=-1)))
    cos = np.array(cos)
    assert np.median(cos) > 0.999 and cos.min() > 0.98
    so, sg = o.stats(), g.stats()
    assert sg["steps"] == so["steps"] and sg["refresh"] == so["refresh"]
    assert abs(sg["reuse"] - so["reuse"]) <= 0.05 * so["steps"]


def test_forced_fallback_equals_exact_topk_decode(rt, P, oracle_mod):
    """tau > 1: every step is the exact path, so decode_step and exact_topk_decode agree bit for bit."""
    cfg = wl.CONFIGS["tiny"].replace(context=3000, steps=6, B=2, H_q=8, H_kv=2, d=128)
    st = wl.make_stream(cfg, steps=6)
    g = rt.ReTopK.from_config(cfg, tau=2.0, R=0)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    for t in range(6):
        q = P.to_dev(st.q[t])
        a = g.decode_step(q, k, v, st.seq_len(t))
        idx = torch.empty((cfg.B, cfg.H_q, cfg.K), dtype=torch.int32, device="cuda")
        b = g.exact_topk_decode(q, k, v, st.seq_len(t), idx_out=idx)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        assert torch.equal(g.last_step()["support"], idx)
    s = g.stats()
    assert s["fallback"] == 6 * cfg.B * cfg.H_q and s["reuse"] == 0


def test_hand_trace_decisions_on_gpu(rt, P):
    """The six-step hand trace, zero-padded to d = 64 (decisions and supports only)."""
    with open(os.path.join(GOLDEN, "hand_trace.json")) as f:
        gold = json.load(f)
    p = gold["params"]
    d = 64
    keys = np.zeros((1, 1, len(gold["keys"]), d), dtype=np.float32)
    keys[0, 0, :, :2] = np.array(gold["keys"], dtype=np.float32)
    vals = np.zeros_like(keys)
    vals[0, 0, :, :2] = np.array(gold["values"], dtype=np.float32)
    k, v = P.to_dev(bits(keys)), P.to_dev(bits(vals))
    g = rt.ReTopK(1, 1, 1, d, p["M"], p["r"], p["W"], p["K"], p["tau"], p["R"], keys.shape[2])
    names = {"REUSE": 0, "FALLBACK": 1, "REFRESH": 2}
    for t, step in enumerate(gold["steps"]):
        q = np.zeros((1, 1, d), dtype=np.float32)
        q[0, 0, :2] = step["q"]
        g.decode_step(P.to_dev(bits(q)), k, v, step["L"])
        last = g.last_step()
        assert int(last["path"][0, 0]) == names[step["path"]], f"step {t}"
        assert last["support"][0, 0].tolist() == step["support"], f"step {t}"
        if step["candidates"] is not None:
            assert int(last["n_cand"][0, 0]) == len(step["candidates"])
    s = g.stats()
    assert {key: s[key] for key in gold["stats"]} == gold["stats"]


def test_steps_are_deterministic(rt, P):
    cfg = wl.CONFIGS["tiny"].replace(context=4000, steps=20, B=2, H_q=8, H_kv=2, d=128)
    st = wl.make_stream(cfg, steps=20)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    runs = []
    for _ in range(2):
        g = rt.ReTopK.from_config(cfg)
        outs = [g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t)).clone() for t in range(20)]
        runs.append((torch.stack(outs), g.export_state(), g.stats()))
    assert torch.equal(runs[0][0].view(torch.int16), runs[1][0].view(torch.int16))
    assert torch.equal(runs[0][1][0], runs[1][1][0]) and torch.equal(runs[0][1][1], runs[1][1][1])
    assert runs[0][2] == runs[1][2]


@pytest.mark.parametrize("pinned", [True, False])
def test_host_entry_point_matches_device_entry_point(rt, P, pinned):
    """Pinned buffers are read and written by the kernels directly, pageable ones are staged."""
    cfg = wl.CONFIGS["tiny"].replace(context=1500, steps=10, B=2, H_q=8, H_kv=2, d=128)
    st = wl.make_stream(cfg, steps=10)
    g_dev, g_host = rt.ReTopK.from_config(cfg), rt.ReTopK.from_config(cfg)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    # the host path appends each token's key / value itself: start from the prefill only
    k2, v2 = k.clone(), v.clone()
    k2[:, :, cfg.context:] = 0
    v2[:, :, cfg.context:] = 0
    out_host = torch.empty(g_host.q_shape, dtype=torch.bfloat16)
    if pinned:
        out_host = out_host.pin_memory()
    for t in range(10):
        L = st.seq_len(t)
        a = g_dev.decode_step(P.to_dev(st.q[t]), k, v, L)
        qh = rt.bf16_tensor_from_bits(st.q[t], pin=pinned)
        kn = rt.bf16_tensor_from_bits(st.k[:, :, L - 1], pin=pinned)
        vn = rt.bf16_tensor_from_bits(st.v[:, :, L - 1], pin=pinned)
        g_host.decode_step_host(qh, kn, vn, k2, v2, L, out_host)
        assert torch.equal(a.cpu().view(torch.int16), out_host.view(torch.int16))
        assert g_host.last_launch_count() == (4 if pinned else 3)
    assert torch.equal(k, k2) and torch.equal(v, v2)


def test_corrupt_imported_support_is_flagged_not_followed(rt, P):
    cfg = wl.CONFIGS["tiny"].replace(context=500, steps=4)
    st = wl.make_stream(cfg, steps=4)
    g = rt.ReTopK.from_config(cfg, tau=-2.0)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    g.decode_step(P.to_dev(st.q[0]), k, v, st.seq_len(0))
    qbar, sup, n_ins, t_dec = g.export_state()
    sup[0, 0, 0, :5] = 10 ** 6          # far beyond seq_len
    g.import_state(qbar, sup, n_ins, t_dec)
    out = g.decode_step(P.to_dev(st.q[1]), k, v, st.seq_len(1))
    assert torch.isfinite(out.float()).all()
    s = g.stats()
    assert s["status"] & rt.STATUS_BAD_INDEX
    assert int(g.last_step()["support"].max()) < st.seq_len(1)


def test_bad_arguments_return_errors(rt, P):
    g = rt.ReTopK(1, 2, 1, 64, 4, 2, 8, 16, 0.9, 0, 256)
    q = torch.zeros(g.q_shape, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(g.kv_shape, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt.RetopkError):
        g.decode_step(q, kv, kv, 0)
    with pytest.raises(rt.RetopkError):
        g.decode_step(q, kv, kv, 257)
    with pytest.raises(rt.RetopkError):
        rt.ReTopK(1, 2, 1, 64, 4, 5, 8, 16, 0.9, 0, 256)     # r > M


# ------------------------------------------------------------------ prefill seeding

def test_prefill_seeding_matches_oracle(rt, P, oracle_mod):
    """Caches seeded from the last M prompt positions, then free-running decode steps."""
    cfg = wl.CONFIGS["tiny"].replace(context=3000, steps=12, B=2, H_q=8, H_kv=2, d=128, M=8, K=128)
    st = wl.make_stream(cfg, steps=12)
    rng = np.random.default_rng(5)
    n_tail = cfg.M
    q_tail = bits(rng.standard_normal((n_tail, cfg.B, cfg.H_q, cfg.d)))
    # make the prompt's last query equal the first decode query: the first step can then reuse
    q_tail[-1] = st.q[0]
    o = oracle_mod.Oracle.from_config(cfg)
    g = rt.ReTopK.from_config(cfg)
    k, v = P.to_dev(st.k), P.to_dev(st.v)
    o.prefill(q_tail, st.k, st.v, cfg.context)
    g.prefill(P.to_dev(q_tail), k, v, cfg.context)
    assert g.last_launch_count() == 3 * n_tail
    qo, so, n_o, t_o = o.export_state()
    qg, sg, n_g, t_g = g.export_state()
    assert (n_g, t_g) == (n_o, t_o) == (n_tail, 0)
    np.testing.assert_allclose(qg.cpu().numpy(), qo, atol=2e-6)
    sg = sg.cpu().numpy()
    G = cfg.H_q // cfg.H_kv
    for j in range(n_tail):
        L = cfg.context - n_tail + j + 1
        for b in range(cfg.B):
            for h in range(cfg.H_q):
                q64 = wl.bf16_bits_to_f64(q_tail[j, b, h])
                kth = (wl.bf16_bits_to_f64(st.k[b, h // G, so[b, h, j]]) @ q64 / np.sqrt(cfg.d)).min()
                P.assert_support_matches(sg[b, h, j], so[b, h, j], q_tail[j, b, h], st.k[b, h // G], kth,
                                         f"entry {j} seq {b} head {h}")
                assert sg[b, h, j].max() < L
    assert sum(v for key, v in g.stats().items() if key != "status") == 0     # seeding counts nothing
    ex = P.teacher_forced_run(cfg, st, 12, o, g, k, v)
    first_paths = None
    assert o.stats()["reuse"] > 0
    for key in ("steps", "refresh"):
        assert g.stats()[key] == o.stats()[key]


def test_prefill_argument_checks(rt, P):
    g = rt.ReTopK(1, 2, 1, 64, 4, 2, 8, 16, 0.9, 0, 256)
    kv = torch.zeros(g.kv_shape, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt.RetopkError):
        g.prefill(torch.zeros((5, 1, 2, 64), dtype=torch.bfloat16, device="cuda"), kv, kv, 100)   # n_tail > M
    with pytest.raises(rt.RetopkError):
        g.prefill(torch.zeros((3, 1, 2, 64), dtype=torch.bfloat16, device="cuda"), kv, kv, 2)     # n_tail > prompt


def test_recent_recall_variant_teacher_forced(rt, P, oracle_mod):
    """The Recent-R ablation row: newest entries recalled, rho_max over them only."""
    cfg = wl.CONFIGS["tiny"].replace(context=900, steps=30, B=2, H_q=4, H_kv=2, M=6, r=3)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, 30)
    o.set_recall_mode(1)
    g.set_recall_mode(1)
    P.teacher_forced_run(cfg, st, 30, o, g, k, v)
    so, sg = o.stats(), g.stats()
    for key in ("steps", "reuse", "fallback", "refresh", "cand_sum"):
        assert sg[key] == so[key], key
    # and it really differs from similarity recall on this stream
    st2, o2, g2, _, _ = stream_case(rt, P, oracle_mod, cfg, 30)
    for t in range(30):
        o2.decode_step(st2.q[t], st2.k, st2.v, st2.seq_len(t))
    assert o2.stats()["fallback"] != so["fallback"] or o2.stats()["cand_sum"] != so["cand_sum"]


def test_last_recall_reports_the_most_similar_slots(rt, P, oracle_mod):
    """retopk_last_recall against similarities recomputed in fp64 from the oracle's cache (Eq. 6-7)."""
    cfg = wl.CONFIGS["tiny"].replace(context=600, steps=28, B=2, H_q=4, H_kv=2, M=8, r=3)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, cfg.steps)
    same_as_oracle = 0
    for t in range(cfg.steps):
        qbar, sup, n_ins, t_dec = o.export_state()
        g.import_state(torch.from_numpy(qbar.astype(np.float32)).cuda(), torch.from_numpy(sup).cuda(), n_ins, t_dec)
        g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t))
        o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        sel = g.last_recall().cpu().numpy()
        fill = min(n_ins, cfg.M)
        q = wl.bf16_bits_to_f64(st.q[t])
        rho = np.einsum("bhmd,bhd->bhm", qbar, q) / np.linalg.norm(q, axis=-1)[..., None]
        for b in range(cfg.B):
            for h in range(cfg.H_q):
                got = sel[b, h]
                n_sel = min(cfg.r, fill)
                assert (got[n_sel:] == -1).all() and (got[:n_sel] >= 0).all() and (got[:n_sel] < fill).all()
                assert len(set(got[:n_sel])) == n_sel
                if n_sel == 0:
                    continue
                r_sorted = np.sort(rho[b, h, :fill])[::-1]
                mine = rho[b, h, got[:n_sel]]
                assert (np.diff(mine) <= 1e-5).all()                 # most similar first
                assert (mine >= r_sorted[n_sel - 1] - 1e-5).all()     # and none better left out
                last = o.last_step()
                if last["path"][b, h] == 0:        # the oracle records its recall on reuse steps
                    gaps = -np.diff(r_sorted[:n_sel + 1])
                    if gaps.size == 0 or gaps.min() > 1e-5:
                        assert list(got) == list(last["sel"][b, h])
                        same_as_oracle += 1
    assert same_as_oracle > 0.3 * cfg.steps * cfg.B * cfg.H_q


@pytest.mark.parametrize("d", [64, 128])
def test_bf16_query_cache_teacher_forced(rt, P, oracle_mod, d):
    """The bf16 storage variant of the cached queries on both sides."""
    cfg = wl.CONFIGS["tiny"].replace(context=1200, steps=36, B=2, H_q=4, H_kv=2, d=d, M=8, r=3)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, cfg.steps)
    o.set_qbar_format(1)
    g.set_qbar_format(1)
    P.teacher_forced_run(cfg, st, cfg.steps, o, g, k, v)
    so, sg = o.stats(), g.stats()
    assert so["reuse"] > 0 and so["fallback"] > 0
    for key in ("steps", "reuse", "fallback", "refresh", "cand_sum"):
        assert sg[key] == so[key], key
    # the entry the last step stored: the same bf16 value on both sides, but for elements whose
    # fp32 quotient lands on the other side of a rounding boundary (one bf16 step at most)
    slot = (cfg.steps - 1) % cfg.M
    mine = g.export_state()[0][:, :, slot].cpu().numpy().astype(np.float64)
    ref = o.export_state()[0][:, :, slot]
    assert np.array_equal(wl.bf16_bits_to_f64(wl.f32_to_bf16_bits(mine.astype(np.float32))), mine)
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)
    assert (np.abs(mine - ref) <= step * 1.0001).all()
    assert (mine == ref).mean() > 0.99


def test_bf16_query_cache_free_running_and_argument_checks(rt, P, oracle_mod):
    cfg = wl.CONFIGS["tiny"].replace(context=800, steps=40, B=2, H_q=4, H_kv=2)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, cfg.steps)
    o.set_qbar_format(1)
    g.set_qbar_format(1)
    g.set_qbar_format(0)
    g.set_qbar_format(1)
    cos = []
    for t in range(cfg.steps):
        out_g = g.decode_step(P.to_dev(st.q[t]), k, v, st.seq_len(t)).float().cpu().numpy().astype(np.float64)
        out_o = o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        cos.append((out_g * out_o).sum(-1) / (np.linalg.norm(out_g, axis=-1) * np.linalg.norm(out_o, axis=-1)))
    assert np.median(np.array(cos)) > 0.999
    so, sg = o.stats(), g.stats()
    assert sg["steps"] == so["steps"] and abs(sg["reuse"] - so["reuse"]) <= 0.05 * so["steps"]
    lib = rt.load()
    assert lib.retopk_set_qbar_format(g.h, 0) == -1          # the cache is not empty any more
    assert lib.retopk_set_qbar_format(None, 1) == -1
    g.reset()
    assert lib.retopk_set_qbar_format(g.h, 2) == -1
    assert lib.retopk_set_qbar_format(g.h, 0) == 0


def test_failed_launch_in_mid_step_is_sticky_until_reset(rt, P, oracle_mod):
    """A launch that fails after the step's first kernel went out leaves the caches half
    advanced: the step and every later one report the failure until the context is reset
    (the failure is injected on the host; no kernel misbehaves)."""
    cfg = wl.CONFIGS["tiny"].replace(B=1, H_q=2, H_kv=1, context=600, steps=12)
    st, o, g, k, v = stream_case(rt, P, oracle_mod, cfg, 12)
    lib = rt.load()
    q = [P.to_dev(st.q[t]) for t in range(12)]
    for t in range(3):
        g.decode_step(q[t], k, v, st.seq_len(t))
    # a failure of the FIRST launch leaves nothing enqueued: the context stays usable
    assert lib.retopk_debug_fail_next_launch(g.h, 1) == 0
    with pytest.raises(rt.RetopkError):
        g.decode_step(q[3], k, v, st.seq_len(3))
    g.decode_step(q[3], k, v, st.seq_len(3))
    assert g.export_state()[2] == 4
    # a failure of the scan or finish launch is sticky
    for which in (2, 3):
        assert lib.retopk_debug_fail_next_launch(g.h, which) == 0
        with pytest.raises(rt.RetopkError):
            g.decode_step(q[4], k, v, st.seq_len(4))
        with pytest.raises(rt.RetopkError):
            g.decode_step(q[4], k, v, st.seq_len(4))
        g.reset()
        torch.cuda.synchronize()
        # after the reset the context runs the stream again and agrees with the oracle
        o.reset()
        P.teacher_forced_run(cfg, st, 8, o, g, k, v)
    assert lib.retopk_debug_fail_next_launch(g.h, 9) == -1
