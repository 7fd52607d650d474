"""Compile the CUDA library in-tree: ``csrc/retopk_api.cu`` -> ``libretopk.so`` (sm_100a)."""
from __future__ import annotations

import fcntl
import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
SRC_DIR = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libretopk.so")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _sources():
    return sorted(os.path.join(SRC_DIR, f) for f in os.listdir(SRC_DIR)
                  if f.endswith((".cu", ".cuh"))) + [os.path.join(os.path.dirname(_PKG), "include", "retopk.h")]


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(s) > built for s in _sources())


def find_nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: cannot build libretopk.so")
    return nvcc


def build(force: bool = False, verbose: bool = False) -> str:
    """Run nvcc if the library is missing or older than its sources; return its path.

    Several processes may call this at once (one rank per GPU): the check and the build run
    under a file lock, and the library appears under its final name in one rename.
    """
    if not force and not is_stale():
        return LIB_PATH
    nvcc = find_nvcc()
    with open(LIB_PATH + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if force or is_stale():          # another process may have built it meanwhile
                units = [s for s in _sources() if s.endswith(".cu")]
                tmp = f"{LIB_PATH}.{os.getpid()}.tmp"
                cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + units
                subprocess.run(cmd, check=True)
                os.replace(tmp, LIB_PATH)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
