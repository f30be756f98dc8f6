"""The C-ABI library loads and exports every symbol include/slim.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2503_05840_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    return build.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "slim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slim_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib_path):
    L = ctypes.CDLL(lib_path)
    names = _declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(L, n), f"{n} declared in slim.h but not exported"


def test_binding_covers_every_declared_symbol(lib_path):
    assert sorted(binding.SIGNATURES) == _declared_symbols()
    for n in binding.SIGNATURES:
        assert callable(getattr(binding, n)), n


def test_strerror_and_null_argument_checks(lib_path):
    L = binding.lib()
    assert binding.strerror(binding.SLIM_OK) == "ok"
    assert "singular" in binding.strerror(binding.SLIM_ERR_SINGULAR)
    # argument errors are detected before any CUDA call
    assert L.slim_create(None, 64, 2, 32, 0.0, 0) == binding.SLIM_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert L.slim_create(ctypes.byref(h), 64, 2, 31, 0.0, 0) == binding.SLIM_ERR_UNSUPPORTED   # d != H d_k
    assert L.slim_create(ctypes.byref(h), 64, 2, 32, 0.0, 7) == binding.SLIM_ERR_INVALID_ARG   # dtype
    assert L.slim_create(ctypes.byref(h), -4, 2, 32, 0.0, 0) == binding.SLIM_ERR_INVALID_ARG
    assert L.slim_decode(None, None, None, None, None, None, None) == binding.SLIM_ERR_INVALID_ARG
    assert L.slim_append_k(None, None, None, None, 1, None) == binding.SLIM_ERR_INVALID_ARG
    assert L.slim_cache_bytes(None, 1, 1) == 0
    assert L.slim_workspace_bytes(None, 1, 1) == 0
    assert L.slim_query(None, 0) == -1
