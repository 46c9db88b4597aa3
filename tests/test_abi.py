"""The C-ABI library loads, exports every symbol include/bitdelta.h declares, and rejects bad
arguments before touching a device (no compute calls here)."""
import ctypes
import os
import re

import pytest

import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import binding
from paper_2609_36800_b200 import build as bd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    bd_build.build()
    return bd.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bitdelta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bitdelta_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(lib):
    for code in range(0, 10):
        assert bd.status_string(code) != "unknown status"
    assert bd.status_string(99) == "unknown status"


def test_argument_errors_are_reported_without_a_launch(lib):
    p = ctypes.c_void_p
    ok = p(0x1000)   # never dereferenced: argument checks come first
    # NULL pointers
    assert lib.bitdelta_gemm(p(0), ok, ok, ok, ok, 1, 1, 128, 128, ok, 1 << 30, None) == 1
    assert lib.bitdelta_pack(p(0), ok, 1, 1, 32, None) == 1
    # shapes
    assert lib.bitdelta_gemm(ok, ok, ok, ok, ok, 0, 1, 128, 128, ok, 1 << 30, None) == 2
    assert lib.bitdelta_gemm(ok, ok, ok, ok, ok, 1, 1, 128, 100, ok, 1 << 30, None) == 2
    assert lib.bitdelta_pack(ok, ok, 1, 1, 33, None) == 2
    assert lib.bitdelta_unpack(ok, ok, 1, -1, 32, None) == 2
    # alignment
    assert lib.bitdelta_gemm(p(0x1008), ok, ok, ok, ok, 1, 1, 128, 128, ok, 1 << 30, None) == 3
    assert lib.bitdelta_pack(p(0x1001), ok, 1, 1, 32, None) == 3
    assert lib.bitdelta_workspace_init(p(0), 16, None) == 1


def test_workspace_size_query(lib):
    assert bd.gemm_workspace_bytes(0, 1, 128, 128) == 0
    assert bd.gemm_workspace_bytes(1, 1, 128, 100) == 0
    for (B, m, N, K) in [(1, 16, 512, 512), (8, 1, 4096, 4096), (16, 4, 11008, 4096), (4, 512, 4096, 4096),
                         (32, 8, 4096, 14336)]:
        n = bd.gemm_workspace_bytes(B, m, N, K)
        assert 0 < n < (1 << 30)
        assert bd.gemm_host_arena_bytes(B, m, N, K) > n
    assert bd.gemm_workspace_bytes(2, 3, 96, 96) > 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libbitdelta.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()
