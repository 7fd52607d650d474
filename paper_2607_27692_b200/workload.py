"""Seeded synthetic decode streams for ReTopK (inputs only; none of the method's arithmetic).

Both the CPU oracle tests and the CUDA parity tests / benchmark read their inputs from
here, so the two sides always see bit-identical bf16 arrays.  Nothing in this module
scores, selects or attends: it only draws random numbers.

Recipe (per sequence ``b`` and KV head ``g``; all draws from counter-based Philox streams
keyed by ``(seed, stream id)``):

* cluster centres ``c_j ~ N(0, 4 I_d)``, ``n_clusters`` of them;
* every position ``i`` (prefill and decode alike): with probability 0.25 the key is
  ``c_j + 0.5 N(0, I_d)`` for a uniformly drawn ``j``, otherwise ``N(0, I_d)``; values are
  ``N(0, I_d)``; both rounded once to bf16 (round to nearest even);
* queries per (sequence, query head): ``q_0`` uniform on the unit sphere, then
  ``q_t = normalise(a q_{t-1} + s xi_t)`` with ``xi_t`` a uniformly random unit vector,
  except that with probability ``p_jump`` the query jumps to ``c_j / |c_j|`` for a uniform
  centre ``j`` of its KV head; emitted queries are rounded to bf16, the walk itself runs
  in fp64;
* the stress configuration alternates every 16 steps between a calm regime
  ``(a, s, p_jump) = (0.9, 0.44, 0.02)`` and a turbulent one ``(0.6, 0.8, 0.3)``.

bf16 arrays are carried as ``uint16`` bit patterns (numpy has no bf16 type).
"""
from __future__ import annotations

import concurrent.futures as _cf
import dataclasses
import os

import numpy as np

BASE_SEED = 260727692

# Stream-kind tags folded into the Philox key so tensors never share random numbers.
_KIND_CENTRES, _KIND_KEYS, _KIND_VALUES, _KIND_QUERIES = 1, 2, 3, 4


@dataclasses.dataclass(frozen=True)
class Config:
    """One decode workload: shapes, ReTopK hyper-parameters and generator settings."""

    name: str
    config_id: int
    B: int
    H_q: int
    H_kv: int
    d: int
    context: int          # prefilled keys before the first decode step
    steps: int            # decode steps in a full run
    K: int
    M: int
    r: int
    W: int
    tau: float
    R: int
    n_clusters: int
    p_jump: float
    ar: float = 0.9
    noise: float = 0.44
    regime_switch: int = 0   # >0: alternate calm / turbulent every this many steps

    @property
    def max_seq_len(self) -> int:
        return self.context + self.steps

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def cap(self) -> int:
        return self.r * self.K + self.W

    def replace(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "tiny": Config("tiny", 1, 1, 1, 1, 64, 2048, 64, 64, 16, 2, 32, 0.85, 16, 8, 0.05),
    "llama16k": Config("llama16k", 2, 1, 32, 8, 128, 16384, 256, 512, 64, 4, 128, 0.9, 32, 64, 0.02),
    "batch32k": Config("batch32k", 3, 8, 32, 8, 128, 32768, 256, 512, 64, 4, 128, 0.9, 32, 64, 0.02),
    "batch64k": Config("batch64k", 3, 8, 32, 8, 128, 65536, 256, 512, 64, 4, 128, 0.9, 32, 64, 0.02),
    "headline128k": Config("headline128k", 4, 4, 32, 8, 128, 131072, 512, 512, 128, 4, 256, 0.9, 32,
                           256, 0.02),
    # the paper's cross-model setting at 128K uses K = 1024 (Table 2); same streams as the headline
    "headline128k_k1024": Config("headline128k_k1024", 4, 4, 32, 8, 128, 131072, 512, 1024, 128, 4, 256, 0.9, 32,
                                 256, 0.02),
    # one sequence at 128K: the batch size of the paper's own latency measurements
    "single128k": Config("single128k", 6, 1, 32, 8, 128, 131072, 512, 512, 128, 4, 256, 0.9, 32, 256, 0.02),
    "stress128k": Config("stress128k", 5, 16, 32, 8, 128, 131072, 256, 2048, 128, 8, 512, 0.95, 8,
                         256, 0.02, regime_switch=16),
}

_TURBULENT = (0.6, 0.8, 0.3)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def _rng(seed: int, kind: int, a: int, b: int = 0) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64((kind << 48) | (a << 24) | b)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def sequence_seed(cfg: Config, sequence_id: int, layer: int = 0) -> int:
    return BASE_SEED + 1000 * cfg.config_id + sequence_id + 100 * layer


def _centres(cfg: Config, seed: int, g: int) -> np.ndarray:
    return 2.0 * _rng(seed, _KIND_CENTRES, g).standard_normal((cfg.n_clusters, cfg.d))


def _fill_kv_head(cfg: Config, seed: int, g: int, n_pos: int, k_out: np.ndarray, v_out: np.ndarray):
    centres = _centres(cfg, seed, g).astype(np.float32)
    rk = _rng(seed, _KIND_KEYS, g)
    rv = _rng(seed, _KIND_VALUES, g)
    block = 32768
    for lo in range(0, n_pos, block):
        n = min(block, n_pos - lo)
        noise = rk.standard_normal((n, cfg.d), dtype=np.float32)
        near = rk.random(n) < 0.25
        which = rk.integers(0, cfg.n_clusters, size=n)
        keys = np.where(near[:, None], centres[which] + np.float32(0.5) * noise, noise)
        k_out[lo:lo + n] = f32_to_bf16_bits(keys)
        v_out[lo:lo + n] = f32_to_bf16_bits(rv.standard_normal((n, cfg.d), dtype=np.float32))


def _query_walk(cfg: Config, seed: int, h: int, steps: int) -> np.ndarray:
    g = h // cfg.G
    centres = _centres(cfg, seed, g)
    rq = _rng(seed, _KIND_QUERIES, h)
    q = rq.standard_normal(cfg.d)
    q /= np.linalg.norm(q)
    out = np.empty((steps, cfg.d), dtype=np.float32)
    for t in range(steps):
        if t > 0:
            ar, noise, p_jump = cfg.ar, cfg.noise, cfg.p_jump
            if cfg.regime_switch and (t // cfg.regime_switch) % 2 == 1:
                ar, noise, p_jump = _TURBULENT
            xi = rq.standard_normal(cfg.d)
            xi /= np.linalg.norm(xi)
            jump = rq.random() < p_jump
            j = int(rq.integers(0, cfg.n_clusters))
            if jump:
                q = centres[j] / np.linalg.norm(centres[j])
            else:
                q = ar * q + noise * xi
                q /= np.linalg.norm(q)
        out[t] = q
    return out


@dataclasses.dataclass
class Stream:
    """bf16 bit patterns of one layer's decode stream.

    ``k`` / ``v``: ``[B, H_kv, max_seq_len, d]``; ``q``: ``[steps, B, H_q, d]``.
    Decode step ``t`` (0-based) sees ``seq_len = context + t + 1`` keys: the key/value of
    the current token is already in place at position ``context + t``.
    """

    cfg: Config
    k: np.ndarray
    v: np.ndarray
    q: np.ndarray

    def seq_len(self, t: int) -> int:
        return self.cfg.context + t + 1


def make_stream(cfg: Config, steps: int | None = None, layer: int = 0,
                sequences: range | None = None, workers: int | None = None) -> Stream:
    """Generate one layer's K/V cache and query stream for ``cfg``.

    ``steps`` may shorten the run (the KV arrays keep the full ``cfg.max_seq_len`` layout
    so strides match the full workload).  ``sequences`` restricts generation to a subset
    of batch rows (the result then has ``B = len(sequences)``), which full-size parity
    tests use to check sampled sequences one by one.
    """
    steps = cfg.steps if steps is None else steps
    if steps > cfg.steps:
        raise ValueError("steps exceeds the configured run length")
    seqs = list(range(cfg.B)) if sequences is None else list(sequences)
    n_pos = cfg.context + steps
    k = np.zeros((len(seqs), cfg.H_kv, cfg.max_seq_len, cfg.d), dtype=np.uint16)
    v = np.zeros_like(k)
    q = np.empty((steps, len(seqs), cfg.H_q, cfg.d), dtype=np.uint16)

    def kv_job(args):
        bi, b, g = args
        _fill_kv_head(cfg, sequence_seed(cfg, b, layer), g, n_pos, k[bi, g], v[bi, g])

    def q_job(args):
        bi, b, h = args
        q[:, bi, h, :] = f32_to_bf16_bits(_query_walk(cfg, sequence_seed(cfg, b, layer), h, steps))

    workers = workers or min(32, os.cpu_count() or 1)
    with _cf.ThreadPoolExecutor(max_workers=workers) as pool:
        list(pool.map(kv_job, [(bi, b, g) for bi, b in enumerate(seqs) for g in range(cfg.H_kv)]))
        list(pool.map(q_job, [(bi, b, h) for bi, b in enumerate(seqs) for h in range(cfg.H_q)]))
    sub = cfg if sequences is None else cfg.replace(B=len(seqs))
    return Stream(sub, k, v, q)
