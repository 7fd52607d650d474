"""The C interface from a plain C program (run with -m gpu): compiled with gcc against
include/retopk.h and the CUDA runtime, linked to the in-tree library, run as a child process."""
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plain_c_program_drives_the_library(tmp_path):
    from paper_2607_27692_b200 import build
    lib = build.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "decode_from_c")
    cmd = ["gcc", "-std=c99", "-O1", "-o", exe, os.path.join(ROOT, "tests", "c_abi", "decode_from_c.c"),
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           lib, "-L", os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.dirname(lib),
           "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    assert shutil.which("gcc")
    subprocess.run(cmd, check=True)
    res = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip().endswith("OK"), res.stdout + res.stderr
