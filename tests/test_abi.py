"""The C-ABI library builds, loads and exports every symbol include/b2gemm.h declares; host-side argument
checks and the tile selector work without a GPU (nothing here launches a kernel)."""
import ctypes
import json
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def declared_symbols():
    text = (ROOT / "include" / "b2gemm.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(b2_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(b2):
    lib = b2.lib()
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in b2gemm.h but not exported"
    assert sorted(b2.EXPORTED_SYMBOLS) == names, "binding and header disagree on the entry points"


def test_version_and_strerror(b2):
    assert "sm_100a" in b2.version()
    assert b2.strerror(0) == "success"
    assert "8" in b2.strerror(-8)
    assert b2.strerror(1003).startswith("workspace")


def test_argument_checks_need_no_gpu(b2):
    lib = b2.lib()
    d = ctypes.c_double
    fake = ctypes.c_void_p(4096)  # never dereferenced: every call below fails its argument check first

    def dgemm(ta, tb, m, n, k, lda, ldb, ldc, A=fake, B=fake, C=fake):
        return lib.b2_dgemm(ta, tb, m, n, k, d(1.0), A, lda, B, ldb, d(0.0), C, ldc, None)

    assert dgemm(b"X", b"N", 2, 2, 2, 2, 2, 2) == -1
    assert dgemm(b"N", b"Q", 2, 2, 2, 2, 2, 2) == -2
    assert dgemm(b"N", b"N", -1, 2, 2, 2, 2, 2) == -3
    assert dgemm(b"N", b"N", 2, -1, 2, 2, 2, 2) == -4
    assert dgemm(b"N", b"N", 2, 2, -1, 2, 2, 2) == -5
    assert dgemm(b"N", b"N", 2, 2, 2, 2, 2, 2, A=None) == -7
    assert dgemm(b"N", b"N", 3, 2, 2, 2, 2, 3) == -8
    assert dgemm(b"T", b"N", 3, 2, 4, 3, 4, 3) == -8
    assert dgemm(b"N", b"N", 2, 2, 2, 2, 2, 2, B=None) == -9
    assert dgemm(b"N", b"N", 2, 2, 3, 2, 2, 2) == -10
    assert dgemm(b"N", b"T", 2, 3, 2, 2, 2, 2) == -10
    assert dgemm(b"N", b"N", 2, 2, 2, 2, 2, 2, C=None) == -12
    assert dgemm(b"N", b"N", 3, 2, 2, 3, 2, 2) == -13
    # empty problems return success without touching anything
    assert dgemm(b"N", b"N", 0, 2, 2, 1, 2, 1, A=None, B=None, C=None) == 0
    assert dgemm(b"N", b"N", 2, 0, 2, 2, 2, 2, A=None, B=None, C=None) == 0
    assert lib.b2_dgemm_variant(77, b"N", b"N", 2, 2, 2, d(1.0), fake, 2, fake, 2, d(0.0), fake, 2, None) == 1004
    al = (d * 2)(1.0, 0.0)
    assert lib.b2_zgemm4m(b"X", b"N", 2, 2, 2, al, fake, 2, fake, 2, al, fake, 2, fake, 0, None) == -1
    assert lib.b2_zgemm4m(b"N", b"N", 2, 2, 2, None, fake, 2, fake, 2, al, fake, 2, fake, 0, None) == -6
    assert lib.b2_zgemm4m(b"N", b"N", 2, 2, 2, al, fake, 2, fake, 2, None, fake, 2, fake, 0, None) == -11
    assert lib.b2_zgemm4m(b"N", b"N", 2, 2, 2, al, fake, 1, fake, 2, al, fake, 2, fake, 0, None) == -8
    assert lib.b2_zgemm4m(b"N", b"N", 2, 2, 2, al, fake, 2, fake, 2, al, fake, 2, None, 0, None) == 1003
    assert lib.b2_dgemm_host(b"N", b"N", 2, 2, 2, d(1.0), fake, 2, fake, 2, d(0.0), fake, 2, None, 0, None) == 1003
    per = d(0)
    assert lib.b2_pipe_probe(99, 128, 1, 10, fake, 4096, ctypes.byref(per), None) == -1
    assert lib.b2_pipe_probe(0, 100, 1, 10, fake, 4096, ctypes.byref(per), None) == -2
    assert lib.b2_pipe_probe(0, 128, 1, 10, fake, 8, ctypes.byref(per), None) == -6
    # instruction-mix kinds run a micro-kernel's inner loop and take that micro-kernel's CTA size only
    assert lib.b2_pipe_probe(7, 256, 1, 10, fake, 4096, ctypes.byref(per), None) == -2
    assert lib.b2_pipe_probe(11 | 0x100, 128, 1, 10, fake, 4096, ctypes.byref(per), None) == -2


def test_workspace_sizes(b2):
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 4096, 4096, 4096) == 6 * 4096 * 4096 * 8
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 3, 5, 7) % 256 == 0
    assert b2.b2_zgemm4m_workspace_bytes("X", "N", 3, 5, 7) == 0
    assert b2.b2_zgemm4m_workspace_bytes("C", "N", 3, 5, 7) == b2.b2_zgemm4m_workspace_bytes("T", "N", 3, 5, 7)
    assert b2.b2_zgemm3m_workspace_bytes("N", "N", 4096, 4096, 4096) == 9 * 4096 * 4096 * 8
    # A, B, C, and for large problems a second buffer of C's size (the old values of C arrive last)
    assert b2.b2_gemm_host_workspace_bytes(0, "N", "N", 8192, 8192, 8192) == 4 * 8192 * 8192 * 8
    assert b2.b2_gemm_host_workspace_bytes(0, "N", "N", 1024, 1024, 1024) == 3 * 1024 * 1024 * 8
    assert b2.b2_gemm_host_workspace_bytes(1, "T", "N", 1001, 999, 1003) >= 4 * (1003 * 1001 + 1003 * 999 + 1001 * 999)


def test_variant_tables(b2):
    assert b2.b2_variant_count(0) >= 3 and b2.b2_variant_count(1) >= 2 and b2.b2_variant_count(7) == 0
    names = [b2.b2_variant_name(0, v) for v in range(b2.b2_variant_count(0))]
    assert any(n.startswith("dmma") for n in names) and any(n.startswith("dfma") for n in names)
    assert all(b2.b2_variant_name(1, v).startswith("ffma") for v in range(b2.b2_variant_count(1)))
    assert b2.b2_variant_name(0, 99) is None


def test_selector_is_sane_without_gpu(b2):
    """The analytic tile choice: a tensor-core variant for fp64, FFMA for fp32, grid covers C, and tiny problems
    do not get the largest tile."""
    big = json.loads(b2.b2_gemm_query_config(0, "N", "N", 8192, 8192, 8192, 8192, 8192, 8192))
    tiny = json.loads(b2.b2_gemm_query_config(0, "N", "N", 256, 256, 256, 256, 256, 256))
    for cfg, (m, n) in ((big, (8192, 8192)), (tiny, (256, 256))):
        assert cfg["micro_kernel"].startswith("dmma")
        assert cfg["tiles_m"] * cfg["BM"] >= m and cfg["tiles_n"] * cfg["BN"] >= n
        assert cfg["grid"] == cfg["tiles_m"] * cfg["tiles_n"] * cfg["k_split"]
    assert big["micro_kernel"] == "dmma_tma" and tiny["BM"] * tiny["BN"] <= 32 * 32
    f32 = json.loads(b2.b2_gemm_query_config(1, "N", "T", 4096, 4096, 4096, 4096, 4096, 4096))
    # NT with 16-byte aligned columns: the one case where the TMA-staged fp32 kernel is the measured best
    assert f32["micro_kernel"] == "ffma2_tma" and f32["dtype"] == "f32"
    f32 = json.loads(b2.b2_gemm_query_config(1, "N", "N", 4096, 4096, 4096, 4096, 4096, 4096))
    assert f32["micro_kernel"] == "ffma2"
    # tensor-map coordinates are 32-bit: an extent beyond that keeps the selector off the TMA-staged kernels
    long_k = json.loads(b2.b2_gemm_query_config(0, "N", "N", 4096, 4096, 2 ** 31 + 64, 4096, 2 ** 31 + 64, 4096))
    assert long_k["micro_kernel"] == "dmma"
    f32 = json.loads(b2.b2_gemm_query_config(1, "N", "T", 4096, 4096, 4096, 4097, 4096, 4096))
    assert f32["micro_kernel"] == "ffma2"  # odd leading dimension: no tensor map
    with pytest.raises(b2.B2Error):
        b2.b2_gemm_query_config(0, "N", "N", 8, 8, 8, 4, 8, 8)
    with pytest.raises(b2.B2Error):
        b2.b2_gemm_query_config(5, "N", "N", 8, 8, 8, 8, 8, 8)
