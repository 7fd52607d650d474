"""ctypes front end of the fp64 CPU oracle (``retopk_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg
load this; the CUDA library never does.  ``build()`` compiles the C file with gcc next to
itself; nothing here does arithmetic, it only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import fcntl
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "retopk_oracle.c")
_LIB = os.path.join(_HERE, "libretopk_oracle.so")

PATH_REUSE, PATH_FALLBACK, PATH_REFRESH = 0, 1, 2


def _stale() -> bool:
    return not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)


def build(force: bool = False) -> str:
    """Compile the oracle into ``libretopk_oracle.so`` (skipped when up to date; safe to call
    from several processes at once)."""
    if not force and not _stale():
        return _LIB
    with open(_LIB + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if force or _stale():
                tmp = f"{_LIB}.{os.getpid()}.tmp"
                cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
                       "-o", tmp, _SRC, "-lm"]
                subprocess.run(cmd, check=True)
                os.replace(tmp, _LIB)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        vp, i32, i64, f64 = C.c_void_p, C.c_int, C.c_int64, C.c_double
        lib.oracle_create.argtypes = [C.POINTER(vp)] + [i32] * 8 + [f64, i32, i64]
        lib.oracle_create.restype = i32
        lib.oracle_destroy.argtypes = [vp]
        lib.oracle_destroy.restype = None
        lib.oracle_reset.argtypes = [vp]
        lib.oracle_reset.restype = None
        lib.oracle_decode_step.argtypes = [vp, vp, vp, vp, i64, vp]
        lib.oracle_decode_step.restype = i32
        lib.oracle_exact_topk.argtypes = [vp, vp, vp, vp, i64, vp, vp]
        lib.oracle_exact_topk.restype = i32
        lib.oracle_prefill.argtypes = [vp, vp, vp, vp, i64, i32]
        lib.oracle_prefill.restype = i32
        lib.oracle_set_recall_mode.argtypes = [vp, i32]
        lib.oracle_set_recall_mode.restype = i32
        lib.oracle_set_qbar_format.argtypes = [vp, i32]
        lib.oracle_set_qbar_format.restype = i32
        lib.oracle_stats.argtypes = [vp, vp]
        lib.oracle_stats.restype = None
        lib.oracle_last_step.argtypes = [vp] * 7
        lib.oracle_last_step.restype = None
        lib.oracle_fidelity.argtypes = [vp, vp, vp, vp, i64, vp]
        lib.oracle_fidelity.restype = i32
        lib.oracle_last_candidates.argtypes = [vp, i32, vp]
        lib.oracle_last_candidates.restype = i32
        lib.oracle_export_state.argtypes = [vp] * 5
        lib.oracle_export_state.restype = None
        lib.oracle_import_state.argtypes = [vp, vp, vp, i64, i64]
        lib.oracle_import_state.restype = None
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = i32
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 inputs are passed as uint16 bit patterns")
    return a


class Oracle:
    """fp64 ReTopK state machine for ``B`` sequences x ``H_q`` query heads."""

    def __init__(self, B, H_q, H_kv, d, M, r, W, K, tau, R, max_seq_len):
        self.lib = _load()
        self.B, self.H_q, self.H_kv, self.d = B, H_q, H_kv, d
        self.M, self.r, self.W, self.K, self.R = M, r, W, K, R
        # the C interface of the CUDA library takes tau as a float: compare against the
        # same value here
        self.tau = float(np.float32(tau))
        self.max_seq_len = max_seq_len
        h = C.c_void_p()
        rc = self.lib.oracle_create(C.byref(h), B, H_q, H_kv, d, M, r, W, K, self.tau, R,
                                    max_seq_len)
        if rc != 0:
            raise ValueError(f"oracle_create failed with {rc}")
        self.h = h
        self.nh = B * H_q

    @classmethod
    def from_config(cls, cfg, **override):
        p = dict(B=cfg.B, H_q=cfg.H_q, H_kv=cfg.H_kv, d=cfg.d, M=cfg.M, r=cfg.r, W=cfg.W, K=cfg.K,
                 tau=cfg.tau, R=cfg.R, max_seq_len=cfg.max_seq_len)
        p.update(override)
        return cls(**p)

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.oracle_destroy(self.h)
            self.h = None

    def reset(self):
        self.lib.oracle_reset(self.h)

    def _check_kv(self, k, v):
        shape = (self.B, self.H_kv, self.max_seq_len, self.d)
        if k.shape != shape or v.shape != shape:
            raise ValueError(f"k/v must have shape {shape}, got {k.shape} / {v.shape}")

    def decode_step(self, q, k, v, seq_len) -> np.ndarray:
        q, k, v = _u16(q), _u16(k), _u16(v)
        self._check_kv(k, v)
        out = np.empty((self.B, self.H_q, self.d), dtype=np.float64)
        rc = self.lib.oracle_decode_step(self.h, _ptr(q), _ptr(k), _ptr(v), seq_len, _ptr(out))
        if rc != 0:
            raise ValueError(f"oracle_decode_step failed with {rc}")
        return out

    def exact_topk(self, q, k, v, seq_len):
        q, k, v = _u16(q), _u16(k), _u16(v)
        self._check_kv(k, v)
        out = np.empty((self.B, self.H_q, self.d), dtype=np.float64)
        idx = np.empty((self.B, self.H_q, self.K), dtype=np.int32)
        rc = self.lib.oracle_exact_topk(self.h, _ptr(q), _ptr(k), _ptr(v), seq_len, _ptr(out),
                                        _ptr(idx))
        if rc != 0:
            raise ValueError(f"oracle_exact_topk failed with {rc}")
        return out, idx

    def prefill(self, q_tail, k, v, prompt_len):
        """Seed the caches from the last ``len(q_tail)`` prompt positions (causal Exact Top-K supports)."""
        q_tail, k, v = _u16(q_tail), _u16(k), _u16(v)
        self._check_kv(k, v)
        n_tail = q_tail.shape[0]
        if q_tail.shape != (n_tail, self.B, self.H_q, self.d):
            raise ValueError("q_tail must be [n_tail, B, H_q, d]")
        rc = self.lib.oracle_prefill(self.h, _ptr(q_tail), _ptr(k), _ptr(v), prompt_len, n_tail)
        if rc != 0:
            raise ValueError(f"oracle_prefill failed with {rc}")

    def set_recall_mode(self, mode: int):
        """0: recall the most similar entries (the method); 1: the most recent ones (Recent-R ablation)."""
        if self.lib.oracle_set_recall_mode(self.h, mode) != 0:
            raise ValueError("bad recall mode")

    def set_qbar_format(self, fmt: int):
        """0: cached queries kept in full precision; 1: rounded to bf16 when stored (empty cache only)."""
        if self.lib.oracle_set_qbar_format(self.h, fmt) != 0:
            raise ValueError("bad format, or the cache is not empty")

    def stats(self) -> dict:
        five = np.zeros(5, dtype=np.int64)
        self.lib.oracle_stats(self.h, _ptr(five))
        return dict(zip(("steps", "reuse", "fallback", "refresh", "cand_sum"), map(int, five)))

    def last_step(self) -> dict:
        sup = np.empty((self.B, self.H_q, self.K), dtype=np.int32)
        path = np.empty((self.B, self.H_q), dtype=np.uint8)
        rho = np.empty((self.B, self.H_q), dtype=np.float64)
        ncand = np.empty((self.B, self.H_q), dtype=np.int32)
        kth = np.empty((self.B, self.H_q), dtype=np.float64)
        sel = np.empty((self.B, self.H_q, self.r), dtype=np.int32)
        self.lib.oracle_last_step(self.h, _ptr(sup), _ptr(path), _ptr(rho), _ptr(ncand), _ptr(kth),
                                  _ptr(sel))
        return dict(support=sup, path=path, rho_max=rho, n_cand=ncand, kth_score=kth, sel=sel)

    def fidelity(self, q, k, v, seq_len) -> dict:
        """Fidelity of the step just taken against Exact Top-K on the same inputs (Eq. 2-3, Sec. 4).

        Call right after ``decode_step`` with that step's arguments.  Per (sequence, head):
        ``support_recall``, ``retained_mass``, ``output_cosine`` and ``coverage`` (of the exact
        support by the recalled supports, -1 where the step did not reuse).
        """
        q, k, v = _u16(q), _u16(k), _u16(v)
        self._check_kv(k, v)
        four = np.empty((self.B, self.H_q, 4), dtype=np.float64)
        if self.lib.oracle_fidelity(self.h, _ptr(q), _ptr(k), _ptr(v), seq_len, _ptr(four)) != 0:
            raise ValueError("oracle_fidelity failed")
        return dict(support_recall=four[..., 0], retained_mass=four[..., 1], output_cosine=four[..., 2],
                    coverage=four[..., 3])

    def last_candidates(self, b, h):
        cand = np.empty(self.r * self.K + self.W + 1, dtype=np.int32)
        n = self.lib.oracle_last_candidates(self.h, b * self.H_q + h, _ptr(cand))
        return None if n < 0 else cand[:n].copy()

    def export_state(self):
        qbar = np.empty((self.B, self.H_q, self.M, self.d), dtype=np.float64)
        sup = np.empty((self.B, self.H_q, self.M, self.K), dtype=np.int32)
        n_ins, t_dec = C.c_int64(), C.c_int64()
        self.lib.oracle_export_state(self.h, _ptr(qbar), _ptr(sup), C.byref(n_ins), C.byref(t_dec))
        return qbar, sup, int(n_ins.value), int(t_dec.value)

    def import_state(self, qbar, sup, n_ins, t_dec):
        qbar = np.ascontiguousarray(qbar, dtype=np.float64)
        sup = np.ascontiguousarray(sup, dtype=np.int32)
        assert qbar.shape == (self.B, self.H_q, self.M, self.d)
        assert sup.shape == (self.B, self.H_q, self.M, self.K)
        self.lib.oracle_import_state(self.h, _ptr(qbar), _ptr(sup), n_ins, t_dec)
