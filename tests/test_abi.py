"""The C-ABI library loads and exports every symbol include/ec.h declares, and
rejects bad arguments on the host before any launch (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2203_17063_b200 import build

    path = build.build()
    return C.CDLL(path)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ec_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "ec_allreduce_apply" in names and "ec_allgatherv" in names and "ec_kmeans_iterate" in names
    for name in names:
        assert hasattr(lib, name), name


def test_binding_table_matches_header():
    from paper_2203_17063_b200 import binding

    assert sorted(binding.SYMBOLS) == declared_symbols()


def test_host_side_validation(lib):
    lib.ec_allreduce_workspace_bytes.restype = C.c_size_t
    lib.ec_allreduce_workspace_bytes.argtypes = [C.c_int, C.c_size_t, C.c_size_t]
    assert lib.ec_allreduce_workspace_bytes(16, 1 << 24, 65536) == 2 * 2048
    assert lib.ec_allreduce_workspace_bytes(256, 1 << 20, 8192) == 2 * 4096
    assert lib.ec_allreduce_workspace_bytes(0, 10, 2) == 0
    assert lib.ec_allreduce_workspace_bytes(1025, 10, 2) == 0
    assert lib.ec_allreduce_workspace_bytes(4, 0, 2) == 0
    assert lib.ec_allreduce_workspace_bytes(4, 10, 0) == 0
    lib.ec_allreduce_init.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_size_t,
                                      C.c_int, C.c_void_p, C.c_size_t]
    h = C.c_void_p()
    assert lib.ec_allreduce_init(C.byref(h), 0, 10, 0, 0, 2, 0, None, 0) == -1          # P < 1
    assert lib.ec_allreduce_init(C.byref(h), 4, 10, 9, 0, 2, 0, None, 0) == -1          # dtype
    assert lib.ec_allreduce_init(C.byref(h), 4, 10, 2, 0, 2, 1, None, 0) == -2          # pairwise on int64
    assert lib.ec_allreduce_init(C.byref(h), 4, 10, 0, 1, 2, 1, None, 0) == -2          # pairwise max
    assert lib.ec_allreduce_init(None, 4, 10, 0, 0, 2, 0, None, 0) == -1
    assert lib.ec_allreduce_init(C.byref(h), 4, 10, 0, 0, 2, 0, C.c_void_p(256), 8) == -5   # workspace too small
    lib.ec_allreduce_apply.argtypes = [C.c_void_p] * 2 + [C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_size_t] + [C.c_void_p] * 4
    assert lib.ec_allreduce_apply(None, None, 4, 10, 0, 0, 2, None, None, None, None) == -1
    lib.ec_allgatherv.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_size_t, C.c_void_p, C.c_void_p]
    assert lib.ec_allgatherv(None, None, 4, 2, None, None, None, 0, None, None) == -1
    lib.ec_kmeans_workspace_bytes.restype = C.c_size_t
    lib.ec_kmeans_workspace_bytes.argtypes = [C.c_size_t, C.c_int, C.c_int, C.c_int]
    assert lib.ec_kmeans_workspace_bytes(1000, 30, 4, 2) == 0                            # D % 4 != 0
    assert lib.ec_kmeans_workspace_bytes(1000, 32, 2000, 2) == 0                         # K too large
    lib.ec_strerror.restype = C.c_char_p
    assert lib.ec_strerror(0) == b"ok" and b"invalid" in lib.ec_strerror(-1)
    assert lib.ec_version() >= 1000
