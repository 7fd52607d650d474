"""Shared comparison code for the GPU parity tests (CUDA library vs the fp64 oracle)."""
import math

import numpy as np
import torch

from paper_2607_27692_b200 import retopk as rt
from paper_2607_27692_b200 import workload as wl

ABS_TOL, REL_TOL = 2e-2, 1e-2        # outputs: bf16 I/O, fp32 accumulate
SCORE_BAND = 1e-3                    # relative band around the K-th score
TAU_BAND = 1e-4                      # similarity band around tau


def to_dev(bits):
    return rt.bf16_tensor_from_bits(bits, device="cuda")


def assert_outputs_close(out_gpu, out_ref, what=""):
    g = out_gpu.float().cpu().numpy().astype(np.float64)
    err = np.abs(g - out_ref)
    tol = ABS_TOL + REL_TOL * np.abs(out_ref)
    assert (err <= tol).all(), f"{what}: max err {err.max():.4g} (worst excess {(err - tol).max():.4g})"


def assert_support_matches(sup_gpu, sup_ref, q_bits, k_head_bits, kth_score, what=""):
    """Index sets must agree except for positions scoring within the band of the K-th score."""
    sg, sr = sup_gpu[sup_gpu >= 0], sup_ref[sup_ref >= 0]
    assert len(sg) == len(sr), f"{what}: support sizes differ ({len(sg)} vs {len(sr)})"
    assert (np.diff(sg) > 0).all(), f"{what}: GPU support not strictly ascending"
    diff = np.setxor1d(sg, sr)
    if len(diff) == 0:
        return 0
    q64 = wl.bf16_bits_to_f64(q_bits)
    s = wl.bf16_bits_to_f64(k_head_bits[diff]) @ q64 / math.sqrt(len(q64))
    band = SCORE_BAND * max(abs(kth_score), 1e-30)
    assert (np.abs(s - kth_score) <= band).all(), (
        f"{what}: {len(diff)} positions differ, worst gap {np.abs(s - kth_score).max():.3g} "
        f"vs band {band:.3g}")
    return len(diff)


def synthetic_full_state(oracle, st, L0, rng, n_inserted=None, spread=0.35, dup_slots=()):
    """A cache that is full before the first step: written into the oracle (import it into the
    GPU context from there).  Cached queries are noisy unit-norm copies of the stream's first
    queries (so that similarities spread around typical thresholds), supports are sorted random
    index sets below ``L0``.  ``dup_slots``: pairs (a, b) of slots made identical, which ties
    their similarities exactly.  ``n_inserted`` >= M places the ring's write position."""
    B, H, M, d, K = oracle.B, oracle.H_q, oracle.M, oracle.d, oracle.K
    q0 = wl.bf16_bits_to_f64(st.q[0])                       # [B, H, d]
    q0 = q0 / np.maximum(np.linalg.norm(q0, axis=-1, keepdims=True), 1e-30)
    qbar = q0[:, :, None, :] + spread * rng.standard_normal((B, H, M, d)) / np.sqrt(d) * np.linspace(0.2, 4.0, M)[None, None, :, None]
    qbar /= np.linalg.norm(qbar, axis=-1, keepdims=True)
    sup = np.empty((B, H, M, K), dtype=np.int32)
    for b in range(B):
        for h in range(H):
            for c in range(M):
                n = min(K, L0)
                row = np.sort(rng.choice(L0, size=n, replace=False)).astype(np.int32)
                sup[b, h, c, :n] = row
                sup[b, h, c, n:] = -1
    for a, b_ in dup_slots:
        qbar[:, :, b_] = qbar[:, :, a]
    if oracle_is_bf16(oracle):
        qbar = wl.bf16_bits_to_f64(wl.f32_to_bf16_bits(qbar.astype(np.float32)))
    oracle.import_state(qbar, sup, M + M // 2 if n_inserted is None else n_inserted, 0)


def oracle_is_bf16(oracle):
    return bool(getattr(oracle, "qbar_bf16", False))


def teacher_forced_run(cfg, st, steps, oracle, gpu, k_dev, v_dev, b_map=None, check_out=True,
                       full_stream=None, check_candidates=True):
    """Step both sides with the GPU caches re-seeded from the oracle before every step.

    ``oracle`` may cover a subset of the GPU's sequences: ``b_map[i]`` is the GPU batch row of
    oracle row ``i`` (the stream ``st`` then holds the oracle's rows, ``full_stream`` the
    queries of every GPU sequence).  With ``check_candidates`` the candidate list (Eq. 9) of
    every head that reuses is compared element by element.  Returns counts of excused events.
    """
    G = cfg.H_q // cfg.H_kv
    b_map = list(range(oracle.B)) if b_map is None else b_map
    full = len(b_map) == gpu.B
    excused_flips = excused_pos = 0
    q_full = None
    if check_candidates:
        gpu.debug_candidates(True)
    for t in range(steps):
        L = st.seq_len(t)
        qbar, sup, n_ins, t_dec = oracle.export_state()
        if full:
            gq = torch.from_numpy(qbar.astype(np.float32)).cuda()
            gs = torch.from_numpy(sup).cuda()
        else:
            gq, gs, _, _ = gpu.export_state()
            idx = torch.tensor(b_map, device="cuda")
            gq[idx] = torch.from_numpy(qbar.astype(np.float32)).cuda()
            gs[idx] = torch.from_numpy(sup).cuda()
        gpu.import_state(gq, gs, n_ins, t_dec)
        if full:
            q_dev = to_dev(st.q[t])
        elif full_stream is not None:
            q_dev = to_dev(full_stream.q[t])
        else:
            q_full = torch.zeros(gpu.q_shape, dtype=torch.bfloat16, device="cuda") if q_full is None else q_full
            q_full[torch.tensor(b_map, device="cuda")] = to_dev(st.q[t])
            q_dev = q_full
        out_g = gpu.decode_step(q_dev, k_dev, v_dev, L)
        out_o = oracle.decode_step(st.q[t], st.k, st.v, L)
        lo, lg = oracle.last_step(), gpu.last_step()
        g_path = lg["path"].cpu().numpy()
        g_sup = lg["support"].cpu().numpy()
        g_rho = lg["rho_max"].cpu().numpy()
        g_nc = lg["n_cand"].cpu().numpy()
        g_cand = gpu.last_candidates().cpu().numpy() if check_candidates else None
        for i, b in enumerate(b_map):
            for h in range(cfg.H_q):
                what = f"step {t} seq {b} head {h}"
                rho_o = lo["rho_max"][i, h]
                if np.isfinite(rho_o):
                    assert abs(g_rho[b, h] - rho_o) <= 2e-5, f"{what}: rho_max {g_rho[b, h]} vs {rho_o}"
                else:
                    assert g_rho[b, h] == rho_o
                if g_path[b, h] != lo["path"][i, h]:
                    assert abs(rho_o - oracle.tau) <= TAU_BAND, (
                        f"{what}: path {g_path[b, h]} vs {lo['path'][i, h]}, rho_max {rho_o}")
                    excused_flips += 1
                    continue
                if lo["path"][i, h] == 0:
                    assert g_nc[b, h] == lo["n_cand"][i, h], f"{what}: n_cand"
                    if check_candidates:
                        want = oracle.last_candidates(i, h)
                        assert np.array_equal(g_cand[b, h, :len(want)], want), f"{what}: candidate list"
                excused_pos += assert_support_matches(
                    g_sup[b, h], lo["support"][i, h], st.q[t, i, h], st.k[i, h // G],
                    lo["kth_score"][i, h], what)
                if check_out:
                    assert_outputs_close(out_g[b, h], out_o[i, h], what)
    return dict(flips=excused_flips, positions=excused_pos)
