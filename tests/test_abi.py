"""The C interface loads and exports what include/retopk.h declares (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_27692_b200 import build, retopk
    build.build()
    return retopk.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "retopk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(retopk_\w+|exact_topk_\w+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2607_27692_b200 import retopk
    names = declared_functions()
    assert "retopk_decode_step" in names and "exact_topk_decode" in names and len(names) >= 12
    for name in names:
        assert hasattr(lib, name), f"{name} declared in retopk.h but not exported"
    assert set(names) == set(retopk.SIGNATURES), "binding and header disagree"


def test_error_strings_and_argument_checks(lib):
    assert lib.retopk_strerror(0) == b"ok"
    assert b"invalid" in lib.retopk_strerror(-1)
    h = C.c_void_p()
    # rejected before any CUDA call: r > M, H_q not a multiple of H_kv, K < 1
    assert lib.retopk_create_batched(C.byref(h), 1, 4, 2, 128, 2, 3, 8, 16, 0.9, 0, 1024) == -1
    assert lib.retopk_create_batched(C.byref(h), 1, 5, 2, 128, 4, 2, 8, 16, 0.9, 0, 1024) == -1
    assert lib.retopk_create_batched(C.byref(h), 1, 4, 2, 128, 4, 2, 8, 0, 0.9, 0, 1024) == -1
    # legal but unsupported head dim
    assert lib.retopk_create_batched(C.byref(h), 1, 4, 2, 96, 4, 2, 8, 16, 0.9, 0, 1024) == -2
    assert h.value is None
    assert lib.retopk_decode_step(None, None, None, None, 1, None, None) == -1
    assert lib.retopk_destroy(None) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2607_27692_b200 import retopk
    monkeypatch.setattr(retopk, "_lib", None)
    monkeypatch.setattr(retopk, "library_path", lambda: str(tmp_path / "nope.so"))
    with pytest.raises(retopk.RetopkError):
        retopk.load()
