"""CPU-only checks of the boundary: the library builds and loads, and exports
every symbol the header declares (no compute calls without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sidco.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2101_10761_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sidco_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_compress_entry_point():
    syms = declared_symbols()
    assert "sidco_compress" in syms and "sidco_compress_host" in syms and len(syms) >= 12


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} declared in sidco.h but not exported"


def test_binding_lists_the_same_symbols():
    from paper_2101_10761_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    for name in binding.EXPORTS:
        assert hasattr(binding, name)


def test_host_only_entry_points(lib):
    lib.sidco_version.restype = ctypes.c_int
    assert lib.sidco_version() >= 100
    lib.sidco_error_string.restype = ctypes.c_char_p
    lib.sidco_error_string.argtypes = [ctypes.c_int]
    assert b"delta" in lib.sidco_error_string(-3)
    lib.sidco_workspace_bytes.restype = ctypes.c_size_t
    lib.sidco_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int]
    small, big = lib.sidco_workspace_bytes(1000, 1), lib.sidco_workspace_bytes(25557032, 161)
    assert 0 < small < big
    assert 12 * 25557032 < big < 13 * 25557032       # staging (index, value) and the side values dominate
    lib.sidco_set_params.argtypes = [ctypes.c_double] * 3 + [ctypes.c_int]
    assert lib.sidco_set_params(0.25, 0.2, 0.2, 5) == 0
    assert lib.sidco_set_params(1.5, 0.2, 0.2, 5) == -6
    assert lib.sidco_set_params(0.25, 0.2, 0.2, 0) == -6


def test_argument_errors_are_found_before_any_cuda_call(lib):
    i64 = ctypes.c_int64
    off = (i64 * 3)(0, 4, 8)
    bad = (i64 * 3)(0, 5, 4)
    vp = ctypes.c_void_p
    lib.sidco_compress.argtypes = [vp, vp, ctypes.POINTER(i64), ctypes.c_int, ctypes.c_float, ctypes.c_int,
                                   ctypes.c_int, vp, vp, vp, vp]
    p = 0x1000  # never dereferenced: every call below fails validation first
    assert lib.sidco_compress(None, p, off, 2, 0.1, 0, 1, p, p, p, None) == -1
    assert lib.sidco_compress(p, p + 64, bad, 2, 0.1, 0, 1, p, p, p, None) == -2
    assert lib.sidco_compress(p, p + 64, off, 0, 0.1, 0, 1, p, p, p, None) == -2
    assert lib.sidco_compress(p, p + 64, off, 2, 0.0, 0, 1, p, p, p, None) == -3
    assert lib.sidco_compress(p, p + 64, off, 2, 1.0, 0, 1, p, p, p, None) == -3
    assert lib.sidco_compress(p, p + 64, off, 2, 0.1, 3, 1, p, p, p, None) == -4
    assert lib.sidco_compress(p, p + 64, off, 2, 0.1, 0, 0, p, p, p, None) == -5
    assert lib.sidco_compress(p, p + 64, off, 2, 0.1, 0, 9, p, p, p, None) == -5
    assert lib.sidco_compress(p, p + 16, off, 2, 0.1, 0, 1, p, p, p, None) == -9
