"""Pins for the fp64 oracle: every check compares it with something that is not itself.

Brute force (numpy sort), a library routine (torch scaled-dot-product attention), closed
forms, the paper's invariants and a hand-enumerated trace.  None of these needs a GPU.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from paper_2607_27692_b200 import workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
PATHS = {"REUSE": 0, "FALLBACK": 1, "REFRESH": 2}


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def brute_topk(q64, k64, K):
    """Indices of the K largest q.k/sqrt(d): full sort on (score desc, index asc)."""
    s = (k64 @ q64) / math.sqrt(q64.shape[0])
    order = np.lexsort((np.arange(len(s)), -s))
    return np.sort(order[:K]), s


def softmax_v(s, idx, v64):
    w = np.exp(s[idx] - s[idx].max())
    return (w[:, None] * v64[idx]).sum(0) / w.sum()


def random_case(seed, B, H_q, H_kv, d, L, Lmax):
    rng = np.random.default_rng(seed)
    k = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    v = bits(rng.standard_normal((B, H_kv, Lmax, d)))
    q = bits(rng.standard_normal((B, H_q, d)))
    return q, k, v


# ------------------------------------------------------------------ Exact Top-K (Eq. 1, 4, 12)

@pytest.mark.parametrize("H_q,H_kv,d,L,K", [(1, 1, 64, 300, 17), (4, 2, 32, 1000, 64),
                                             (8, 2, 128, 513, 512), (2, 1, 16, 50, 50)])
def test_exact_topk_matches_brute_force(oracle_mod, H_q, H_kv, d, L, K):
    B, Lmax = 2, L + 7
    q, k, v = random_case(10 + L, B, H_q, H_kv, d, L, Lmax)
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, K, 0.85, 0, Lmax)
    out, idx = o.exact_topk(q, k, v, L)
    G = H_q // H_kv
    for b in range(B):
        for h in range(H_q):
            k64 = wl.bf16_bits_to_f64(k[b, h // G, :L])
            v64 = wl.bf16_bits_to_f64(v[b, h // G, :L])
            q64 = wl.bf16_bits_to_f64(q[b, h])
            want, s = brute_topk(q64, k64, K)
            assert np.array_equal(idx[b, h], want)
            # selected scores dominate the rest
            rest = np.setdiff1d(np.arange(L), want)
            if len(rest):
                assert s[want].min() >= s[rest].max()
            np.testing.assert_allclose(out[b, h], softmax_v(s, want, v64), rtol=1e-12, atol=1e-13)


def test_k_at_least_L_is_dense_attention(oracle_mod):
    """With K >= L the exact support is every key, so Eq. 12 is ordinary softmax attention."""
    B, H_q, H_kv, d, L = 2, 4, 2, 64, 200
    q, k, v = random_case(3, B, H_q, H_kv, d, L, L)
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 2, 8, L + 5, 0.85, 0, L)
    out, idx = o.exact_topk(q, k, v, L)
    assert np.array_equal(idx[..., :L], np.broadcast_to(np.arange(L), (B, H_q, L)))
    assert (idx[..., L:] == -1).all()
    tq = torch.from_numpy(wl.bf16_bits_to_f64(q)).reshape(B, H_q, 1, d)
    tk = torch.from_numpy(wl.bf16_bits_to_f64(k)).repeat_interleave(H_q // H_kv, dim=1)
    tv = torch.from_numpy(wl.bf16_bits_to_f64(v)).repeat_interleave(H_q // H_kv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).reshape(B, H_q, d)
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_k1_returns_value_of_best_key(oracle_mod):
    B, H_q, H_kv, d, L = 1, 2, 1, 32, 400
    q, k, v = random_case(5, B, H_q, H_kv, d, L, L)
    o = oracle_mod.Oracle(B, H_q, H_kv, d, 4, 1, 0, 1, 0.85, 0, L)
    out, idx = o.exact_topk(q, k, v, L)
    for h in range(H_q):
        s = wl.bf16_bits_to_f64(k[0, 0]) @ wl.bf16_bits_to_f64(q[0, h])
        assert idx[0, h, 0] == int(np.argmax(s))
        np.testing.assert_array_equal(out[0, h], wl.bf16_bits_to_f64(v[0, 0, idx[0, h, 0]]))


def test_two_keys_logistic_closed_form(oracle_mod):
    d = 4
    q = bits([[[1.0, 2.0, -1.0, 0.5]]])
    k = bits([[[[0.5, 0.25, 1.0, 2.0], [1.0, -1.0, 0.5, 0.0]]]])
    v = bits([[[[1.0, 0.0, 2.0, -4.0], [3.0, 8.0, -2.0, 0.5]]]])
    o = oracle_mod.Oracle(1, 1, 1, d, 1, 1, 0, 2, 0.5, 0, 2)
    out, _ = o.exact_topk(q, k, v, 2)
    e0 = (0.5 + 0.5 - 1.0 + 1.0) / 2.0
    e1 = (1.0 - 2.0 - 0.5) / 2.0
    p0 = 1.0 / (1.0 + math.exp(e1 - e0))
    want = p0 * np.array([1.0, 0.0, 2.0, -4.0]) + (1 - p0) * np.array([3.0, 8.0, -2.0, 0.5])
    np.testing.assert_allclose(out[0, 0], want, rtol=1e-14)


def test_exact_ties_take_lowest_index(oracle_mod):
    """Integer-valued inputs give exact score ties; the lower index must win."""
    d, L, K = 4, 64, 10
    rng = np.random.default_rng(0)
    kf = rng.integers(-2, 3, size=(1, 1, L, d)).astype(np.float32)
    kf[0, 0, 7] = 0.0
    kf[0, 0, 9] = -0.0          # signed zero must tie with +0.0 scores
    qf = np.array([[[1.0, -1.0, 2.0, 0.0]]], dtype=np.float32)
    q, k, v = bits(qf), bits(kf), bits(rng.standard_normal((1, 1, L, d)))
    o = oracle_mod.Oracle(1, 1, 1, d, 1, 1, 0, K, 0.5, 0, L)
    _, idx = o.exact_topk(q, k, v, L)
    s = kf[0, 0].astype(np.float64) @ qf[0, 0].astype(np.float64)
    assert len(np.unique(s)) < L // 2          # the case really has many ties
    order = sorted(range(L), key=lambda i: (-s[i], i))
    assert np.array_equal(idx[0, 0], np.sort(order[:K]))


# ------------------------------------------------------------------ whole ReTopK step

def run_stream(oracle_mod, cfg, steps, **override):
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg, **override)
    return st, o


def test_tau_above_one_is_exact_every_step(oracle_mod):
    """Check (a): when no similarity can reach tau, every step is the Exact Top-K path."""
    cfg = wl.CONFIGS["tiny"].replace(context=256, steps=24)
    st, o = run_stream(oracle_mod, cfg, 24, tau=2.0, R=0)
    for t in range(24):
        L = st.seq_len(t)
        out = o.decode_step(st.q[t], st.k, st.v, L)
        ref, idx = o.exact_topk(st.q[t], st.k, st.v, L)
        last = o.last_step()
        assert (last["path"] == oracle_mod.PATH_FALLBACK).all()
        assert np.array_equal(last["support"], idx)
        np.testing.assert_array_equal(out, ref)
    assert o.stats()["fallback"] == 24 and o.stats()["reuse"] == 0


def test_window_covering_history_recovers_exact_support(oracle_mod):
    """Check (b): if the candidate set contains S_t, reranking returns S_t exactly."""
    cfg = wl.CONFIGS["tiny"].replace(context=200, steps=20, H_q=4, H_kv=2)
    st = wl.make_stream(cfg, steps=20)
    o = oracle_mod.Oracle.from_config(cfg, tau=-2.0, R=0, W=cfg.max_seq_len)
    for t in range(20):
        L = st.seq_len(t)
        out = o.decode_step(st.q[t], st.k, st.v, L)
        ref, idx = o.exact_topk(st.q[t], st.k, st.v, L)
        last = o.last_step()
        want = oracle_mod.PATH_FALLBACK if t == 0 else oracle_mod.PATH_REUSE
        assert (last["path"] == want).all()
        if t > 0:
            assert (last["n_cand"] == L).all()
        assert np.array_equal(last["support"], idx)
        np.testing.assert_allclose(out, ref, rtol=1e-13, atol=1e-15)


def test_hand_trace(oracle_mod):
    """Check (c): six steps enumerated by hand (insert / evict, fallback, refresh, ties)."""
    with open(os.path.join(GOLDEN, "hand_trace.json")) as f:
        g = json.load(f)
    p = g["params"]
    keys = np.array(g["keys"], dtype=np.float32)
    vals = np.array(g["values"], dtype=np.float32)
    Lmax = len(keys)
    k = bits(keys.reshape(1, 1, Lmax, 2))
    v = bits(vals.reshape(1, 1, Lmax, 2))
    o = oracle_mod.Oracle(p["B"], p["H_q"], p["H_kv"], p["d"], p["M"], p["r"], p["W"], p["K"],
                          p["tau"], p["R"], Lmax)
    for t, step in enumerate(g["steps"]):
        assert step["L"] == g["prefill"] + t + 1
        q = bits(np.array(step["q"], dtype=np.float32).reshape(1, 1, 2))
        out = o.decode_step(q, k, v, step["L"])
        last = o.last_step()
        assert last["path"][0, 0] == PATHS[step["path"]], f"step {t}"
        known = [x for x in step["rho"] if x is not None]
        if known:
            assert last["rho_max"][0, 0] == pytest.approx(max(known), abs=1e-12)
        else:
            assert last["rho_max"][0, 0] == -np.inf
        assert list(last["support"][0, 0]) == step["support"], f"step {t}"
        if step["candidates"] is not None:
            assert list(o.last_candidates(0, 0)) == step["candidates"]
        # Eq. 12 with two selected keys is a logistic mix of their values
        a, b = step["support"]
        ea, eb = (step["qk"][str(a)] / math.sqrt(2.0), step["qk"][str(b)] / math.sqrt(2.0))
        pa = 1.0 / (1.0 + math.exp(eb - ea))
        want = pa * vals[a].astype(np.float64) + (1 - pa) * vals[b].astype(np.float64)
        np.testing.assert_allclose(out[0, 0], want, rtol=1e-13)
        # ring slot written by this step
        qbar, sup, n_ins, t_dec = o.export_state()
        assert n_ins == t + 1 and t_dec == t + 1
        assert list(sup[0, 0, step["slot"]]) == step["support"]
        qn = np.array(step["q"], dtype=np.float64)
        np.testing.assert_allclose(qbar[0, 0, step["slot"]], qn / np.linalg.norm(qn), rtol=1e-15)
    assert o.stats() == g["stats"]


def test_capacity_example_from_paper(oracle_mod):
    """Eq. 14 upper bound is attained by disjoint supports: 4*512 + 32 = 2080."""
    with open(os.path.join(GOLDEN, "hand_trace.json")) as f:
        ex = json.load(f)["capacity_example"]
    r, K, W = ex["r"], ex["K"], ex["W"]
    M, d, L = r, 8, 4096
    o = oracle_mod.Oracle(1, 1, 1, d, M, r, W, K, -2.0, 0, L)
    qbar = np.zeros((1, 1, M, d))
    qbar[0, 0, :, 0] = 1.0
    sup = np.stack([np.arange(K) + 600 * c for c in range(M)]).astype(np.int32).reshape(1, 1, M, K)
    o.import_state(qbar, sup, M, 1)
    rng = np.random.default_rng(1)
    q = bits(np.abs(rng.standard_normal((1, 1, d))) + 0.1)
    k = bits(rng.standard_normal((1, 1, L, d)))
    v = bits(rng.standard_normal((1, 1, L, d)))
    o.decode_step(q, k, v, L)
    last = o.last_step()
    assert last["path"][0, 0] == oracle_mod.PATH_REUSE
    assert last["n_cand"][0, 0] == ex["capacity"] == r * K + W
    # duplicates collapse: identical recalled supports give |support U window|
    sup2 = np.broadcast_to(sup[0, 0, 0], (1, 1, M, K)).copy()
    o.import_state(qbar, sup2, M, 1)
    o.decode_step(q, k, v, L)
    assert o.last_step()["n_cand"][0, 0] == K + W
    cand = o.last_candidates(0, 0)
    assert (np.diff(cand) > 0).all()


@pytest.mark.parametrize("name,override", [
    ("tiny", {}),
    ("tiny", {"r": 1}),
    ("tiny", {"M": 1, "r": 1}),
    ("tiny", {"W": 0}),
    ("tiny", {"R": 0}),
    ("tiny", {"tau": -2.0}),
])
def test_invariants_on_streams(oracle_mod, name, override):
    """Counter identities, the candidate bounds of Eq. 14 and the rerank guarantees."""
    steps = 40
    cfg = wl.CONFIGS[name].replace(context=512, steps=steps, H_q=2, H_kv=1, B=2)
    st = wl.make_stream(cfg, steps=steps)
    o = oracle_mod.Oracle.from_config(cfg, **override)
    K, r, W, R = o.K, o.r, o.W, o.R
    tau = o.tau
    seen_reuse = 0
    for t in range(steps):
        L = st.seq_len(t)
        o.decode_step(st.q[t], st.k, st.v, L)
        _, exact_idx = o.exact_topk(st.q[t], st.k, st.v, L)
        last = o.last_step()
        for b in range(cfg.B):
            for h in range(cfg.H_q):
                path = last["path"][b, h]
                sup = last["support"][b, h]
                assert (sup >= 0).all() and (np.diff(sup) > 0).all() and sup.max() < L
                refresh_due = R > 0 and t > 0 and t % R == 0
                if refresh_due:
                    assert path == oracle_mod.PATH_REFRESH
                elif last["rho_max"][b, h] < tau:
                    assert path == oracle_mod.PATH_FALLBACK
                else:
                    assert path == oracle_mod.PATH_REUSE
                if path == oracle_mod.PATH_REUSE:
                    seen_reuse += 1
                    cand = o.last_candidates(b, h)
                    assert max(K, min(W, L)) <= len(cand) <= r * K + W
                    assert (np.diff(cand) > 0).all()
                    assert np.isin(sup, cand).all()
                    # an exact-support member that was recalled must survive the rerank
                    recalled = np.intersect1d(exact_idx[b, h], cand)
                    assert np.isin(recalled, sup).all()
                    if len(recalled) == K:
                        assert np.array_equal(sup, exact_idx[b, h])
                    if W > 0:
                        assert np.isin(np.arange(max(0, L - W), L), cand).all()
                else:
                    assert np.array_equal(sup, exact_idx[b, h])
    s = o.stats()
    nh = cfg.B * cfg.H_q
    assert s["steps"] == steps * nh == s["reuse"] + s["fallback"] + s["refresh"]
    assert s["refresh"] == ((steps - 1) // R if R > 0 else 0) * nh
    if override.get("tau", 0) <= -1:
        assert s["fallback"] == nh      # only the empty-cache step
    assert seen_reuse == s["reuse"] and seen_reuse > 0


def test_topr_recall_matches_brute_force(oracle_mod):
    """Eq. 7: the recalled slots are the r most similar cached queries."""
    B, H, d, M, r, K, L = 1, 3, 16, 8, 3, 4, 64
    rng = np.random.default_rng(4)
    qc = rng.standard_normal((B, H, M, d))
    qc /= np.linalg.norm(qc, axis=-1, keepdims=True)
    sup = np.sort(rng.permuted(np.tile(np.arange(L), (B, H, M, 1)), axis=-1)[..., :K], axis=-1)
    o = oracle_mod.Oracle(B, H, H, d, M, r, 2, K, -2.0, 0, L)
    o.import_state(qc, sup.astype(np.int32), M + 3, 5)
    q, k, v = random_case(8, B, H, H, d, L, L)
    o.decode_step(q, k, v, L)
    last = o.last_step()
    q64 = wl.bf16_bits_to_f64(q)
    for h in range(H):
        qb = q64[0, h] / np.linalg.norm(q64[0, h])
        rho = qc[0, h] @ qb
        want = sorted(range(M), key=lambda c: (-rho[c], c))[:r]
        assert list(last["sel"][0, h]) == want
        assert last["rho_max"][0, h] == pytest.approx(rho.max(), abs=1e-14)
        cand = o.last_candidates(0, h)
        union = np.union1d(np.unique(sup[0, h, want]), np.arange(L - 2, L))
        assert np.array_equal(cand, union)
    # insert went to ring slot (M + 3) % M and evicted what was there
    qbar, sup_after, n_ins, t_dec = o.export_state()
    assert n_ins == M + 4 and t_dec == 6
    slot = (M + 3) % M
    assert np.array_equal(sup_after[0, 0, slot], last["support"][0, 0])
    untouched = [c for c in range(M) if c != slot]
    assert np.array_equal(sup_after[0, :, untouched], sup[0][:, untouched].transpose(1, 0, 2))


def test_short_history_pads_support(oracle_mod):
    """Fewer keys than K: select what exists, pad with -1, never index out of range."""
    d, K, L = 8, 16, 5
    q, k, v = random_case(2, 1, 1, 1, d, L, 32)
    o = oracle_mod.Oracle(1, 1, 1, d, 2, 1, 3, K, -2.0, 0, 32)
    o.decode_step(q, k, v, L)
    sup = o.last_step()["support"][0, 0]
    assert list(sup[:L]) == list(range(L)) and (sup[L:] == -1).all()
    out = o.decode_step(q, k, v, L + 1)
    last = o.last_step()
    assert last["path"][0, 0] == oracle_mod.PATH_REUSE and last["n_cand"][0, 0] == L + 1
    assert np.isfinite(out).all()


def test_similarity_equal_to_tau_reuses(oracle_mod):
    """Eq. 13 falls back only for rho_max strictly below tau."""
    d, L = 4, 16
    rng = np.random.default_rng(9)
    k = bits(rng.standard_normal((1, 1, L, d)))
    v = bits(rng.standard_normal((1, 1, L, d)))
    o = oracle_mod.Oracle(1, 1, 1, d, 2, 1, 2, 4, 1.0, 0, L)
    e0 = bits(np.array([[[2.0, 0.0, 0.0, 0.0]]]))      # normalises to exactly (1,0,0,0)
    e1 = bits(np.array([[[0.0, 3.0, 0.0, 0.0]]]))
    want = [oracle_mod.PATH_FALLBACK, oracle_mod.PATH_REUSE, oracle_mod.PATH_FALLBACK]
    for t, q in enumerate([e0, e0, e1]):
        o.decode_step(q, k, v, 10 + t)
        assert o.last_step()["path"][0, 0] == want[t]
    assert o.last_step()["rho_max"][0, 0] == 0.0


# ------------------------------------------------------------------ prefill seeding (Sec. 3.3)

def test_prefill_seeds_causal_exact_supports(oracle_mod):
    """Each of the last n_tail prompt positions p enters with q/|q| and Top-K over keys 0..p."""
    B, H_q, H_kv, d, M, K, P, n_tail = 1, 4, 2, 16, 6, 5, 40, 4
    rng = np.random.default_rng(21)
    k = bits(rng.standard_normal((B, H_kv, 64, d)))
    v = bits(rng.standard_normal((B, H_kv, 64, d)))
    q_tail = bits(rng.standard_normal((n_tail, B, H_q, d)))
    o = oracle_mod.Oracle(B, H_q, H_kv, d, M, 2, 3, K, 0.5, 0, 64)
    o.prefill(q_tail, k, v, P)
    qbar, sup, n_ins, t_dec = o.export_state()
    assert n_ins == n_tail and t_dec == 0
    for j in range(n_tail):
        L = P - n_tail + j + 1
        for h in range(H_q):
            q64 = wl.bf16_bits_to_f64(q_tail[j, 0, h])
            want, _ = brute_topk(q64, wl.bf16_bits_to_f64(k[0, h // 2, :L]), K)
            assert np.array_equal(sup[0, h, j], want)
            assert sup[0, h, j].max() < L                       # causal: nothing beyond its own position
            np.testing.assert_allclose(qbar[0, h, j], q64 / np.linalg.norm(q64), rtol=1e-15)
    assert (sup[0, :, n_tail:] == -1).all()
    assert sum(o.stats().values()) == 0                         # seeding is not a decode step


def test_prefilled_cache_lets_the_first_step_reuse(oracle_mod):
    """With a seeded cache the first decode step is no longer a forced fallback."""
    cfg = wl.CONFIGS["tiny"].replace(context=300, steps=8, H_q=2, H_kv=1)
    st = wl.make_stream(cfg, steps=8)
    n_tail = cfg.M
    # the prompt's last queries: the stream's first query repeated keeps every similarity at 1
    q_tail = np.broadcast_to(st.q[0], (n_tail,) + st.q[0].shape).copy()
    o = oracle_mod.Oracle.from_config(cfg, R=0)
    o.prefill(q_tail, st.k, st.v, cfg.context)
    for t in range(8):
        o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        if t == 0:
            last = o.last_step()
            assert (last["path"] == oracle_mod.PATH_REUSE).all()
            assert np.allclose(last["rho_max"], 1.0, atol=1e-12)
    s = o.stats()
    assert s["reuse"] >= 2 and s["refresh"] == 0
    # without seeding the first step of every head falls back
    o2 = oracle_mod.Oracle.from_config(cfg, R=0)
    o2.decode_step(st.q[0], st.k, st.v, st.seq_len(0))
    assert (o2.last_step()["path"] == oracle_mod.PATH_FALLBACK).all()


def test_prefill_argument_checks(oracle_mod):
    o = oracle_mod.Oracle(1, 1, 1, 8, 2, 1, 1, 2, 0.5, 0, 16)
    k = bits(np.zeros((1, 1, 16, 8)))
    with pytest.raises(ValueError):
        o.prefill(bits(np.zeros((3, 1, 1, 8))), k, k, 10)      # more tail positions than cache slots
    with pytest.raises(ValueError):
        o.prefill(bits(np.zeros((2, 1, 1, 8))), k, k, 1)       # more tail positions than prompt tokens


# ------------------------------------------------------------------ Recent-R recall (Table 3 ablation row)

def test_recent_recall_takes_the_newest_entries(oracle_mod):
    B, H, d, M, r, K, L = 1, 2, 16, 6, 3, 4, 64
    rng = np.random.default_rng(31)
    qc = rng.standard_normal((B, H, M, d))
    qc /= np.linalg.norm(qc, axis=-1, keepdims=True)
    sup = np.sort(rng.permuted(np.tile(np.arange(L - 4), (B, H, M, 1)), axis=-1)[..., :K], axis=-1).astype(np.int32)
    n_ins = 10                                   # ring of 6: newest entries sit in slots 3, 2, 1
    q, k, v = random_case(9, B, H, H, d, L, L)
    o = oracle_mod.Oracle(B, H, H, d, M, r, 2, K, -2.0, 0, L)
    o.set_recall_mode(1)
    o.import_state(qc, sup, n_ins, 4)
    o.decode_step(q, k, v, L)
    last = o.last_step()
    q64 = wl.bf16_bits_to_f64(q)
    for h in range(H):
        assert list(last["sel"][0, h]) == [3, 2, 1]
        qb = q64[0, h] / np.linalg.norm(q64[0, h])
        assert last["rho_max"][0, h] == pytest.approx((qc[0, h, [3, 2, 1]] @ qb).max(), abs=1e-14)
        union = np.union1d(np.unique(sup[0, h, [3, 2, 1]]), np.arange(L - 2, L))
        assert np.array_equal(o.last_candidates(0, h), union)
    # similarity mode on the same state picks by rho instead
    o2 = oracle_mod.Oracle(B, H, H, d, M, r, 2, K, -2.0, 0, L)
    o2.import_state(qc, sup, n_ins, 4)
    o2.decode_step(q, k, v, L)
    rho = qc[0, 0] @ (q64[0, 0] / np.linalg.norm(q64[0, 0]))
    assert list(o2.last_step()["sel"][0, 0]) == sorted(range(M), key=lambda c: (-rho[c], c))[:r]


def test_recent_recall_falls_back_on_its_own_maximum(oracle_mod):
    """rho_max is taken over the recalled (recent) entries only."""
    d, M, L = 8, 4, 32
    qc = np.zeros((1, 1, M, d))
    qc[0, 0, 0, 0] = 1.0            # old entry identical to the query
    qc[0, 0, 1, 1] = 1.0
    qc[0, 0, 2, 2] = 1.0            # newest two entries are orthogonal to it
    qc[0, 0, 3, 3] = 1.0
    sup = np.tile(np.arange(4, dtype=np.int32), (1, 1, M, 1))
    k = bits(np.random.default_rng(1).standard_normal((1, 1, L, d)))
    q = bits(np.array([[[1.0] + [0.0] * (d - 1)]]))
    for mode, want in ((0, oracle_mod.PATH_REUSE), (1, oracle_mod.PATH_FALLBACK)):
        o = oracle_mod.Oracle(1, 1, 1, d, M, 2, 2, 4, 0.5, 0, L)
        o.set_recall_mode(mode)
        o.import_state(qc, sup, 4, 1)       # ring full: newest are slots 3 and 2
        o.decode_step(q, k, k, 20)
        assert o.last_step()["path"][0, 0] == want


def test_bf16_query_cache_rounds_once_to_nearest(oracle_mod):
    """bf16 storage of the cached queries: every stored element is a bf16 value, the nearest one
    to the fp64 normalised query, and later similarities use the stored values as they are."""
    cfg = wl.CONFIGS["tiny"].replace(context=200, steps=10, H_q=2, H_kv=1, B=2, M=4)
    st = wl.make_stream(cfg, steps=cfg.steps)
    o = oracle_mod.Oracle.from_config(cfg)
    o.set_qbar_format(1)
    off_grid = 0
    for t in range(cfg.steps):
        qbar_before, _, n_ins, _ = o.export_state()
        o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        q = wl.bf16_bits_to_f64(st.q[t])
        exact = q / np.linalg.norm(q, axis=-1, keepdims=True)
        # similarities of this step: unrounded current query against the stored entries
        fill = min(n_ins, cfg.M)
        if fill:
            rho = np.einsum("bhmd,bhd->bhm", qbar_before[:, :, :fill], exact)
            assert np.allclose(o.last_step()["rho_max"], rho.max(-1), rtol=0, atol=1e-13)
        stored = o.export_state()[0][:, :, n_ins % cfg.M]
        # representable: a round trip through the 16-bit pattern changes nothing
        assert np.array_equal(wl.bf16_bits_to_f64(wl.f32_to_bf16_bits(stored.astype(np.float32))), stored)
        # nearest: within half a unit in the last of bf16's 8 significand bits
        ulp = 2.0 ** (np.floor(np.log2(np.abs(exact))) - 7)
        assert (np.abs(stored - exact) <= 0.5 * ulp * (1 + 1e-12)).all()
        off_grid += int((stored != exact).sum())
    assert off_grid > 0.9 * cfg.steps * cfg.B * cfg.H_q * cfg.d      # the rounding really happened


def test_bf16_query_cache_is_off_by_default_and_only_set_on_an_empty_cache(oracle_mod):
    cfg = wl.CONFIGS["tiny"].replace(context=100, steps=3, H_q=1, H_kv=1)
    st = wl.make_stream(cfg, steps=3)
    o = oracle_mod.Oracle.from_config(cfg)
    o.decode_step(st.q[0], st.k, st.v, st.seq_len(0))
    q = wl.bf16_bits_to_f64(st.q[0])
    assert np.allclose(o.export_state()[0][:, :, 0], q / np.linalg.norm(q, axis=-1, keepdims=True), rtol=0, atol=1e-15)
    with pytest.raises(ValueError):
        o.set_qbar_format(1)
    o.reset()
    o.set_qbar_format(1)
    with pytest.raises(ValueError):
        o.set_qbar_format(2)


# ------------------------------------------------------------------ fidelity diagnostics (Eq. 2-3, Sec. 4)
def test_fidelity_on_the_hand_trace(oracle_mod):
    """Step 3 of the hand trace keeps {0,2} where the exact support is {1,2}: recall 1/2,
    coverage 1/2 (the recalled support is {0,2}), retained mass = the logistic weight of key 2
    against key 1 (q.k = 21 vs 16, d = 2).  Steps 1 and 5 rerank to the exact support."""
    with open(os.path.join(GOLDEN, "hand_trace.json")) as f:
        g = json.load(f)
    p = g["params"]
    keys = np.array(g["keys"], dtype=np.float32)
    vals = np.array(g["values"], dtype=np.float32)
    Lmax = len(keys)
    k = bits(keys.reshape(1, 1, Lmax, 2))
    v = bits(vals.reshape(1, 1, Lmax, 2))
    o = oracle_mod.Oracle(p["B"], p["H_q"], p["H_kv"], p["d"], p["M"], p["r"], p["W"], p["K"],
                          p["tau"], p["R"], Lmax)
    seen = {}
    for t, step in enumerate(g["steps"]):
        q = bits(np.array(step["q"], dtype=np.float32).reshape(1, 1, 2))
        o.decode_step(q, k, v, step["L"])
        seen[t] = {name: float(val[0, 0]) for name, val in o.fidelity(q, k, v, step["L"]).items()}
    # exact-path steps reproduce Exact Top-K by construction; coverage is only defined on reuse steps
    for t in (0, 2, 4):
        assert seen[t]["support_recall"] == 1.0 and seen[t]["retained_mass"] == pytest.approx(1.0, abs=1e-15)
        assert seen[t]["output_cosine"] == pytest.approx(1.0, abs=1e-15) and seen[t]["coverage"] == -1.0
    assert seen[1]["support_recall"] == 1.0 and seen[1]["coverage"] == 1.0     # recalled {0,2} = exact {0,2}
    assert seen[3]["support_recall"] == 0.5 and seen[3]["coverage"] == 0.5
    assert seen[3]["retained_mass"] == pytest.approx(1.0 / (1.0 + math.exp((16.0 - 21.0) / math.sqrt(2.0))), rel=1e-13)
    # step 3's output mixes v0, v2 instead of v1, v2: cosine of the two logistic mixes
    v64 = vals.astype(np.float64)
    pa = lambda ea, eb: 1.0 / (1.0 + math.exp((eb - ea) / math.sqrt(2.0)))
    mix = lambda a, b, ea, eb: pa(ea, eb) * v64[a] + (1.0 - pa(ea, eb)) * v64[b]
    got, exact = mix(0, 2, 12.0, 21.0), mix(1, 2, 16.0, 21.0)
    assert seen[3]["output_cosine"] == pytest.approx(
        float(got @ exact / (np.linalg.norm(got) * np.linalg.norm(exact))), rel=1e-12)
    assert seen[5]["support_recall"] == 1.0 and seen[5]["coverage"] == 1.0     # recalled {1,2} = exact {1,2}


def test_fidelity_is_perfect_when_the_window_covers_the_history(oracle_mod):
    """W >= L: the candidates are every key, rerank recovers the exact support, so recall, mass
    and cosine are exactly 1; coverage by the recalled supports alone stays a fraction."""
    cfg = wl.CONFIGS["tiny"].replace(context=300, steps=12, W=400, tau=-2.0, R=0, K=32)
    st = wl.make_stream(cfg)
    o = oracle_mod.Oracle.from_config(cfg)
    for t in range(cfg.steps):
        o.decode_step(st.q[t], st.k, st.v, st.seq_len(t))
        f = o.fidelity(st.q[t], st.k, st.v, st.seq_len(t))
        assert (f["support_recall"] == 1.0).all()
        np.testing.assert_allclose(f["retained_mass"], 1.0, rtol=0, atol=1e-14)
        np.testing.assert_allclose(f["output_cosine"], 1.0, rtol=0, atol=1e-14)
        if t > 0:
            assert ((f["coverage"] >= 0.0) & (f["coverage"] <= 1.0)).all()


def test_fidelity_matches_a_numpy_restatement(oracle_mod):
    """The four quantities recomputed with numpy set operations from the oracle's own step
    record (support, recalled slots, cache state before the step) and a brute-force exact support."""
    cfg = wl.CONFIGS["tiny"].replace(B=2, H_q=4, H_kv=2, context=400, steps=24, K=16, W=8, M=8, r=3, tau=0.5, R=0)
    st = wl.make_stream(cfg)
    o = oracle_mod.Oracle.from_config(cfg)
    G = cfg.H_q // cfg.H_kv
    saw_reuse = False
    for t in range(cfg.steps):
        L = st.seq_len(t)
        _, sup_before, _, _ = o.export_state()
        out = o.decode_step(st.q[t], st.k, st.v, L)
        last = o.last_step()
        f = o.fidelity(st.q[t], st.k, st.v, L)
        for b in range(cfg.B):
            for h in range(cfg.H_q):
                q64 = wl.bf16_bits_to_f64(st.q[t, b, h])
                k64 = wl.bf16_bits_to_f64(st.k[b, h // G, :L])
                v64 = wl.bf16_bits_to_f64(st.v[b, h // G, :L])
                s_exact, scores = brute_topk(q64, k64, cfg.K)
                s_got = set(int(x) for x in last["support"][b, h] if x >= 0)
                w = np.exp(scores[s_exact] - scores[s_exact].max())
                w /= w.sum()
                kept = np.array([i in s_got for i in s_exact])
                assert f["support_recall"][b, h] == pytest.approx(kept.mean(), abs=1e-15)
                assert f["retained_mass"][b, h] == pytest.approx(float(w[kept].sum()), rel=1e-12, abs=1e-15)
                o_exact = w @ v64[s_exact]
                cos = float(out[b, h] @ o_exact / (np.linalg.norm(out[b, h]) * np.linalg.norm(o_exact)))
                assert f["output_cosine"][b, h] == pytest.approx(cos, rel=1e-12)
                if last["path"][b, h] == oracle_mod.PATH_REUSE:
                    saw_reuse = True
                    union = set()
                    for c in last["sel"][b, h]:
                        if c >= 0:
                            union |= set(int(x) for x in sup_before[b, h, c] if x >= 0)
                    cov = np.mean([i in union for i in s_exact])
                    assert f["coverage"][b, h] == pytest.approx(cov, abs=1e-15)
                else:
                    assert f["coverage"][b, h] == -1.0
    assert saw_reuse
