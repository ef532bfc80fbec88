"""The C ABI without a GPU: the library loads, exports what include/llvq.h declares, and the
host-only entry points validate their arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_02652_b200 import binding, build

    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "llvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(llvq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2609_02652_b200 import binding

    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.SYMBOLS) <= set(names)


def test_layout_bytes_and_argument_checks(lib):
    from paper_2609_02652_b200 import binding

    assert binding.layout_bytes(binding.PLANES, 3072, 3072) == 3072 * 128 * 14
    assert binding.layout_bytes(binding.PLANES, 33, 48) == 2 * 2 * 448
    assert binding.layout_bytes(binding.ONEHOT, 8192, 8208) == 8192 * 342 * 20
    n = ctypes.c_size_t()
    assert lib.llvq_layout_bytes(5, 32, 24, ctypes.byref(n)) == -1
    assert lib.llvq_layout_bytes(0, 32, 25, ctypes.byref(n)) == -1
    assert lib.llvq_layout_bytes(0, 0, 24, ctypes.byref(n)) == -1
    assert lib.llvq_gemv_fp16(None, None, None, 8, 8, None) == -1
    assert lib.llvq_gemv(None, 0, None, None, None, None, None, 1, 24, None) == -1
    assert b"aligned" in lib.llvq_strerror(-2)


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2609_02652_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libllvq.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
