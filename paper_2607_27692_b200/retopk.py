"""Python binding of the ReTopK C library (argument marshalling only).

Every step of the decode path runs inside ``libretopk.so``; this module turns torch tensors
into raw pointers and sizes, nothing else.  There is no CPU or PyTorch fallback: if the
library has not been built (``python -m paper_2607_27692_b200.build``) loading fails.

torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

PATH_REUSE, PATH_FALLBACK, PATH_REFRESH = 0, 1, 2
STATUS_BAD_INDEX = 1


class RetopkError(RuntimeError):
    pass


class _Stats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("reuse", C.c_int64), ("fallback", C.c_int64),
                ("refresh", C.c_int64), ("cand_sum", C.c_int64), ("slow_select", C.c_int64), ("scan_groups", C.c_int64),
                ("status", C.c_uint32), ("reserved", C.c_uint32)]


_lib = None

# name -> (restype, argtypes); also the list of symbols include/retopk.h declares
_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
SIGNATURES = {
    "retopk_create": (_i32, [C.POINTER(_vp)] + [_i32] * 7 + [_f32, _i32]),
    "retopk_create_batched": (_i32, [C.POINTER(_vp)] + [_i32] * 8 + [_f32, _i32, _i64]),
    "retopk_set_recall_mode": (_i32, [_vp, _i32]),
    "retopk_set_qbar_format": (_i32, [_vp, _i32]),
    "retopk_set_cluster_size": (_i32, [_vp, _i32]),
    "retopk_set_finish_threads": (_i32, [_vp, _i32]),
    "retopk_set_block_shape": (_i32, [_vp, _i32, _i32]),
    "retopk_set_fusion_level": (_i32, [_vp, _i32, _i32]),
    "retopk_destroy": (_i32, [_vp]),
    "retopk_reset": (_i32, [_vp, _vp]),
    "retopk_decode_step": (_i32, [_vp, _vp, _vp, _vp, _i64, _vp, _vp]),
    "retopk_prefill": (_i32, [_vp, _vp, _vp, _vp, _i64, _i32, _vp]),
    "retopk_decode_step_host": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp]),
    "exact_topk_decode": (_i32, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp]),
    "exact_topk_decode_static": (_i32, [_i32] * 5 + [_i64, _vp, _vp, _vp, _i64, _vp, _vp, _vp]),
    "retopk_stats": (_i32, [_vp, C.POINTER(_Stats)]),
    "retopk_last_step": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "retopk_last_recall": (_i32, [_vp, _vp, _vp]),
    "retopk_debug_candidates": (_i32, [_vp, _i32]),
    "retopk_last_candidates": (_i32, [_vp, _vp, _vp]),
    "retopk_debug_fail_next_launch": (_i32, [_vp, _i32]),
    "retopk_export_state": (_i32, [_vp, _vp, _vp, C.POINTER(_i64), C.POINTER(_i64), _vp]),
    "retopk_import_state": (_i32, [_vp, _vp, _vp, _i64, _i64, _vp]),
    "retopk_profile_begin": (_i32, [_vp, _i32]),
    "retopk_profile_end": (_i32, [_vp, C.POINTER(C.c_double), C.POINTER(_i64)]),
    "retopk_last_launch_count": (_i32, [_vp]),
    "retopk_strerror": (C.c_char_p, [_i32]),
}


def library_path() -> str:
    return _build.LIB_PATH


def load():
    """Load ``libretopk.so`` (must have been built) and declare its signatures."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RetopkError(f"{path} is missing: build it with `python -m paper_2607_27692_b200.build`")
        lib = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise RetopkError(f"{what} failed: {load().retopk_strerror(rc).decode()} ({rc})")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, shape=None) -> int:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"expected a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _host(t: torch.Tensor, dtype, shape) -> int:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise TypeError(f"expected a contiguous host tensor of {dtype} and shape {tuple(shape)}")
    return t.data_ptr()


class ReTopK:
    """One layer's ReTopK context for ``B`` sequences (wraps a ``retopk_ctx*``)."""

    def __init__(self, B, H_q, H_kv, d, M, r, W, K, tau, R, max_seq_len, device="cuda"):
        self.lib = load()
        self.B, self.H_q, self.H_kv, self.d = B, H_q, H_kv, d
        self.M, self.r, self.W, self.K, self.tau, self.R = M, r, W, K, tau, R
        self.max_seq_len = max_seq_len
        self.device = torch.device(device)
        self.h = None
        h = _vp()
        with torch.cuda.device(self.device):
            rc = self.lib.retopk_create_batched(C.byref(h), B, H_q, H_kv, d, M, r, W, K, tau, R,
                                                max_seq_len)
        _check(rc, "retopk_create_batched")
        self.h = h

    @classmethod
    def from_config(cls, cfg, **override):
        p = dict(B=cfg.B, H_q=cfg.H_q, H_kv=cfg.H_kv, d=cfg.d, M=cfg.M, r=cfg.r, W=cfg.W, K=cfg.K,
                 tau=cfg.tau, R=cfg.R, max_seq_len=cfg.max_seq_len)
        p.update(override)
        return cls(**p)

    def close(self):
        if self.h is not None:
            self.lib.retopk_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- shapes ---------------------------------------------------------------------
    @property
    def q_shape(self):
        return (self.B, self.H_q, self.d)

    @property
    def kv_shape(self):
        return (self.B, self.H_kv, self.max_seq_len, self.d)

    # -- calls ----------------------------------------------------------------------
    def set_recall_mode(self, mode: int):
        """0: recall the most similar entries (Eq. 7); 1: the most recent ones (Recent-R ablation row)."""
        _check(self.lib.retopk_set_recall_mode(self.h, mode), "retopk_set_recall_mode")

    def set_qbar_format(self, fmt: int):
        """0: cached queries in fp32 (default); 1: rounded to bf16 when stored (empty cache only)."""
        _check(self.lib.retopk_set_qbar_format(self.h, fmt), "retopk_set_qbar_format")

    def set_cluster_size(self, ctas_per_head: int):
        """CTAs (one SM each) per head in the finish kernel: 1, 2, 4 or 8."""
        _check(self.lib.retopk_set_cluster_size(self.h, ctas_per_head), "retopk_set_cluster_size")

    def set_finish_threads(self, threads: int):
        """Block shape of the finish kernel: 1024 (one CTA per SM) or 512 (two per SM)."""
        _check(self.lib.retopk_set_finish_threads(self.h, threads), "retopk_set_finish_threads")

    def set_block_shape(self, threads: int, ctas_per_sm: int):
        """Block shape of the finish kernel: (1024, 1), (512, 2) or (512, 1)."""
        _check(self.lib.retopk_set_block_shape(self.h, threads, ctas_per_sm), "retopk_set_block_shape")

    def set_fusion_level(self, level: int, dependent_launches: bool = False):
        """Fusion level 1..5 of the reuse path (Table 4's ladder); results do not depend on it."""
        _check(self.lib.retopk_set_fusion_level(self.h, level, int(dependent_launches)), "retopk_set_fusion_level")

    def reset(self):
        _check(self.lib.retopk_reset(self.h, _stream()), "retopk_reset")

    def decode_step(self, q, k_cache, v_cache, seq_len, out=None):
        bf = torch.bfloat16
        if out is None:
            out = torch.empty(self.q_shape, dtype=bf, device=q.device)
        rc = self.lib.retopk_decode_step(self.h, _dev(q, bf, self.q_shape), _dev(k_cache, bf, self.kv_shape),
                                         _dev(v_cache, bf, self.kv_shape), seq_len,
                                         _dev(out, bf, self.q_shape), _stream())
        _check(rc, "retopk_decode_step")
        return out

    def prefill(self, q_tail, k_cache, v_cache, prompt_len):
        """Seed the caches from the last ``len(q_tail)`` prompt positions (q_tail [n_tail,B,H_q,d])."""
        bf = torch.bfloat16
        n_tail = int(q_tail.shape[0])
        rc = self.lib.retopk_prefill(self.h, _dev(q_tail, bf, (n_tail,) + self.q_shape),
                                     _dev(k_cache, bf, self.kv_shape), _dev(v_cache, bf, self.kv_shape),
                                     prompt_len, n_tail, _stream())
        _check(rc, "retopk_prefill")

    def decode_step_host(self, q_host, k_new_host, v_new_host, k_cache, v_cache, seq_len, out_host):
        bf = torch.bfloat16
        kv_new = (self.B, self.H_kv, self.d)
        rc = self.lib.retopk_decode_step_host(
            self.h, _host(q_host, bf, self.q_shape), _host(k_new_host, bf, kv_new),
            _host(v_new_host, bf, kv_new), _dev(k_cache, bf, self.kv_shape),
            _dev(v_cache, bf, self.kv_shape), seq_len, _host(out_host, bf, self.q_shape), _stream())
        _check(rc, "retopk_decode_step_host")
        return out_host

    def exact_topk_decode(self, q, k_cache, v_cache, seq_len, out=None, idx_out=None):
        bf = torch.bfloat16
        if out is None:
            out = torch.empty(self.q_shape, dtype=bf, device=q.device)
        idx_ptr = None if idx_out is None else _dev(idx_out, torch.int32, (self.B, self.H_q, self.K))
        rc = self.lib.exact_topk_decode(self.h, _dev(q, bf, self.q_shape), _dev(k_cache, bf, self.kv_shape),
                                        _dev(v_cache, bf, self.kv_shape), seq_len,
                                        _dev(out, bf, self.q_shape), idx_ptr, _stream())
        _check(rc, "exact_topk_decode")
        return out

    def stats(self) -> dict:
        st = _Stats()
        _check(self.lib.retopk_stats(self.h, C.byref(st)), "retopk_stats")
        return {name: int(getattr(st, name)) for name, _ in _Stats._fields_ if name != "reserved"}

    def last_step(self) -> dict:
        dev = self.device
        sup = torch.empty((self.B, self.H_q, self.K), dtype=torch.int32, device=dev)
        path = torch.empty((self.B, self.H_q), dtype=torch.uint8, device=dev)
        rho = torch.empty((self.B, self.H_q), dtype=torch.float32, device=dev)
        ncand = torch.empty((self.B, self.H_q), dtype=torch.int32, device=dev)
        rc = self.lib.retopk_last_step(self.h, sup.data_ptr(), path.data_ptr(), rho.data_ptr(),
                                       ncand.data_ptr(), _stream())
        _check(rc, "retopk_last_step")
        return dict(support=sup, path=path, rho_max=rho, n_cand=ncand)

    def last_recall(self):
        """Cache slots recalled by the last step (Eq. 7), most similar first, -1 padded: [B, H_q, r] int32."""
        sel = torch.empty((self.B, self.H_q, self.r), dtype=torch.int32, device=self.device)
        _check(self.lib.retopk_last_recall(self.h, sel.data_ptr(), _stream()), "retopk_last_recall")
        return sel

    def debug_candidates(self, enable: bool = True):
        """Test hook: keep the candidate list (Eq. 9) of every head that reuses."""
        _check(self.lib.retopk_debug_candidates(self.h, int(enable)), "retopk_debug_candidates")

    def last_candidates(self):
        """[B, H_q, r*K+W] int32: per reuse head of the last step, its first n_cand entries are the list."""
        cand = torch.empty((self.B, self.H_q, self.r * self.K + self.W), dtype=torch.int32, device=self.device)
        _check(self.lib.retopk_last_candidates(self.h, cand.data_ptr(), _stream()), "retopk_last_candidates")
        return cand

    def export_state(self):
        dev = self.device
        qbar = torch.empty((self.B, self.H_q, self.M, self.d), dtype=torch.float32, device=dev)
        sup = torch.empty((self.B, self.H_q, self.M, self.K), dtype=torch.int32, device=dev)
        n_ins, t_dec = _i64(), _i64()
        rc = self.lib.retopk_export_state(self.h, qbar.data_ptr(), sup.data_ptr(), C.byref(n_ins),
                                          C.byref(t_dec), _stream())
        _check(rc, "retopk_export_state")
        return qbar, sup, int(n_ins.value), int(t_dec.value)

    def import_state(self, qbar, supports, n_inserted, t_dec):
        rc = self.lib.retopk_import_state(
            self.h, _dev(qbar, torch.float32, (self.B, self.H_q, self.M, self.d)),
            _dev(supports, torch.int32, (self.B, self.H_q, self.M, self.K)), n_inserted, t_dec, _stream())
        _check(rc, "retopk_import_state")

    def profile_begin(self, max_calls: int):
        _check(self.lib.retopk_profile_begin(self.h, max_calls), "retopk_profile_begin")

    def profile_end(self) -> dict:
        ms, n = (C.c_double * 3)(), (_i64 * 3)()
        _check(self.lib.retopk_profile_end(self.h, ms, n), "retopk_profile_end")
        return {name: dict(ms=float(ms[i]), launches=int(n[i]))
                for i, name in enumerate(("recall", "scan", "finish"))}

    def last_launch_count(self) -> int:
        return int(self.lib.retopk_last_launch_count(self.h))


STATIC_SCRATCH_BYTES = 32 << 20


def exact_topk_decode_static(q, k_cache, v_cache, seq_len, K, out=None, idx_out=None):
    """Exact Top-K attention through the entry point that allocates nothing.

    For callers that cannot call cudaMalloc (memory owned by another allocator, plug-ins that
    only get buffers): the library's score workspace is a fixed array inside the library
    instead of context memory, so the shape must fit ``STATIC_SCRATCH_BYTES``.  ``out`` and
    ``idx_out`` should be passed in by such callers; they are only created here for
    convenience when omitted.
    """
    bf = torch.bfloat16
    B, H_q, d = q.shape
    _, H_kv, max_seq_len, _ = k_cache.shape
    if out is None:
        out = torch.empty((B, H_q, d), dtype=bf, device=q.device)
    idx_ptr = None if idx_out is None else _dev(idx_out, torch.int32, (B, H_q, K))
    with torch.cuda.device(q.device):
        rc = load().exact_topk_decode_static(
            B, H_q, H_kv, d, K, max_seq_len, _dev(q, bf), _dev(k_cache, bf, (B, H_kv, max_seq_len, d)),
            _dev(v_cache, bf, (B, H_kv, max_seq_len, d)), seq_len, _dev(out, bf, (B, H_q, d)), idx_ptr,
            _stream())
    _check(rc, "exact_topk_decode_static")
    return out


def bf16_tensor_from_bits(bits, device=None, pin=False) -> torch.Tensor:
    """View a numpy ``uint16`` array of bf16 bit patterns as a torch bf16 tensor."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if pin:
        t = t.pin_memory()
    return t if device is None else t.to(device, non_blocking=pin)


def bits_from_bf16_tensor(t: torch.Tensor):
    """bf16 torch tensor -> numpy ``uint16`` bit patterns (host)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
