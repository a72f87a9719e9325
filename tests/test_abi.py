"""The C-ABI library loads and exports every symbol include/rehyat.h declares (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_04342_b200 import build, binding
    build.build()
    return binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rehyat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rehyat_[a-z_]+)\s*\(", text)))


def test_header_declares_the_named_calls():
    names = _declared_symbols()
    for n in ("rehyat_create", "rehyat_forward", "rehyat_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    from paper_2601_04342_b200 import binding
    names = _declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_error_strings_and_null_handling(lib):
    from paper_2601_04342_b200 import binding
    assert lib.rehyat_version() >= 100
    assert lib.rehyat_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert len(lib.rehyat_strerror(code)) > 3
    assert lib.rehyat_destroy(None) == binding.OK
    assert lib.rehyat_workspace_bytes(None) == 0
    # null arguments are rejected before any CUDA call
    h = C.c_void_p(None)
    assert lib.rehyat_create(C.byref(h), None) == binding.ERR_INVALID_ARG
    assert lib.rehyat_create(None, None) == binding.ERR_INVALID_ARG
    # a bad config is rejected before any CUDA call
    cfg = binding.Config(0, 7, 2, 64, 128, 128, 2, 0, 0, 0, 0, 1, 64, 1, 0)
    assert lib.rehyat_create(C.byref(h), C.byref(cfg)) == binding.ERR_INVALID_ARG
    cfg = binding.Config(0, 0, 2, 96, 128, 128, 2, 0, 0, 0, 0, 1, 64, 1, 0)
    assert lib.rehyat_create(C.byref(h), C.byref(cfg)) == binding.ERR_UNSUPPORTED
    cfg = binding.Config(0, 0, 2, 64, 128, 128, 3, 0, 0, 0, 0, 1, 64, 1, 0)   # 128 % 3 != 0
    assert lib.rehyat_create(C.byref(h), C.byref(cfg)) == binding.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2601_04342_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/librehyat.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
