"""The C-ABI library loads without a GPU and exports every symbol include/ralm.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ralm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ralm_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2401_14021_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_paths_calls():
    syms = _declared_symbols()
    for name in ("ralm_index_create", "ralm_index_destroy", "ralm_search", "ralm_cache_search",
                 "ralm_verify", "ralm_device_status", "ralm_status_string"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_status_strings(lib):
    lib.ralm_status_string.restype = ctypes.c_char_p
    seen = {lib.ralm_status_string(i) for i in range(9)}
    assert len(seen) == 9 and all(seen)


def test_host_side_argument_checks_need_no_gpu(lib):
    # every one of these is rejected before any CUDA call
    out = ctypes.c_void_p()
    i64 = ctypes.c_int64
    lib.ralm_index_create.argtypes = [ctypes.c_void_p, i64, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_void_p)]
    INVALID = 1
    assert lib.ralm_index_create(None, 10, 768, 0, 8, 20, ctypes.byref(out)) == INVALID   # null corpus
    assert lib.ralm_index_create(16, 10, 12, 0, 8, 20, ctypes.byref(out)) == INVALID      # d % 8
    assert lib.ralm_index_create(8, 10, 768, 0, 8, 20, ctypes.byref(out)) == INVALID      # misaligned
    assert lib.ralm_index_create(16, -1, 768, 0, 8, 20, ctypes.byref(out)) == INVALID
    assert lib.ralm_index_create(16, 1 << 31, 768, 0, 8, 20, ctypes.byref(out)) == INVALID
    assert lib.ralm_index_create(16, 10, 768, 2, 8, 20, ctypes.byref(out)) == INVALID     # metric
    assert lib.ralm_index_create(16, 10, 768, 0, 0, 20, ctypes.byref(out)) == INVALID
    assert lib.ralm_index_create(16, 10, 768, 0, 8, 2000, ctypes.byref(out)) == INVALID
    assert lib.ralm_index_create(16, 10, 768, 0, 8, 20, None) == INVALID
    assert not out.value
    lib.ralm_verify.argtypes = [ctypes.c_void_p] * 2 + [ctypes.c_int32] * 4 + [ctypes.c_void_p] * 2
    assert lib.ralm_verify(None, None, 4, 3, 1, 1, None, None) == INVALID
    assert lib.ralm_verify(None, None, 4, 3, 1, 2, None, None) == INVALID                 # cmp_k > ld
    assert lib.ralm_verify(None, None, 0, 3, 1, 1, None, None) == 0                       # R == 0
    lib.ralm_search.argtypes = [ctypes.c_void_p] * 2 + [ctypes.c_int32] * 2 + [ctypes.c_void_p] * 3
    assert lib.ralm_search(None, None, 1, 1, None, None, None) == INVALID
    assert lib.ralm_index_destroy(None) == 0


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2401_14021_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_HERE", str(tmp_path))
    with pytest.raises(RuntimeError):
        binding.load_library()
