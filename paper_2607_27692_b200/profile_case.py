"""A few decode steps of ONE layer, for profiler captures of single kernels.

    python -m paper_2607_27692_b200.profile_case CONFIG MODE STEPS

MODE: ``reuse`` (tau = -2: every head reuses after the first step), ``exact`` (tau = 2: every
head takes the full-history path), ``mix`` (the configuration's own tau and refresh period).
One layer keeps the device footprint at a few GB so that a multi-pass capture stays short;
a buffer larger than L2 is rewritten between steps so the key rows come from HBM as they do
in the benchmark's layer rotation.
"""
from __future__ import annotations

import sys

import torch

from . import retopk as rt
from . import workload as wl


def main(argv):
    name, mode, steps = argv[1], argv[2], int(argv[3])
    cfg = wl.CONFIGS[name]
    st = wl.make_stream(cfg, steps=steps)
    k = rt.bf16_tensor_from_bits(st.k, device="cuda")
    v = rt.bf16_tensor_from_bits(st.v, device="cuda")
    q = rt.bf16_tensor_from_bits(st.q, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    override = {"reuse": dict(tau=-2.0, R=0), "exact": dict(tau=2.0, R=0), "mix": {}}[mode]
    ctx = rt.ReTopK.from_config(cfg, **override)
    for t in range(steps):
        flush.zero_()
        ctx.decode_step(q[t], k, v, st.seq_len(t))
    torch.cuda.synchronize()
    print("ok", ctx.stats())


if __name__ == "__main__":
    main(sys.argv)
