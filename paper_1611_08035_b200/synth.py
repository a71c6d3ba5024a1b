"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU-baseline timing.

This module holds no GEMM arithmetic.  Every value is a pure function of (seed, linear
index): a splitmix64 hash of a counter, so the same bytes come out on any device, in any
chunking, and the CPU oracle and the CUDA path can be handed identical data.

Matrices are produced as BLAS storage: a flat tensor of ``ld * cols`` elements, column-major,
``X(r, c) = X[r + c*ld]``.  Rows ``r >= rows`` of every column (the padding ``ld - rows``)
are filled with a poison value (NaN for A and B, a finite sentinel for C) so that a kernel
that reads or writes padding is caught.
"""
from __future__ import annotations

import math

import torch

_MASK64 = (1 << 64) - 1
C_SENTINEL = -7.25e11  # finite, exactly representable in fp32 and fp64, never produced by the test data


def _to_i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GAMMA = _to_i64(0x9E3779B97F4A7C15)
_M1 = _to_i64(0xBF58476D1CE4E5B9)
_M2 = _to_i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def splitmix64(seed: int, index: torch.Tensor) -> torch.Tensor:
    """splitmix64 output for state ``seed + (index+1)*gamma`` (int64 bit patterns, wrapping arithmetic)."""
    z = index * _GAMMA + _to_i64(seed * 0x9E3779B97F4A7C15 + 0x9E3779B97F4A7C15)
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _unit(bits: torch.Tensor) -> torch.Tensor:
    """53-bit uniform in [0, 1) as float64 (exact)."""
    return _lsr(bits, 11).to(torch.float64) * (1.0 / (1 << 53))


def _values(dist: str, seed: int, idx: torch.Tensor) -> torch.Tensor:
    if dist == "uniform":  # i.i.d. uniform on [-1, 1)
        return _unit(splitmix64(seed, idx)) * 2.0 - 1.0
    if dist == "int9":  # integers uniform on {-4, ..., 4}
        r = _lsr(splitmix64(seed, idx), 20) % 9
        return (r - 4).to(torch.float64)
    if dist == "normal":  # standard normal by Box-Muller from two independent streams
        u1 = 1.0 - _unit(splitmix64(seed, idx))  # (0, 1]
        u2 = _unit(splitmix64(seed ^ 0x5DEECE66D, idx))
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    raise ValueError(f"unknown distribution {dist!r}")


def matrix(rows: int, cols: int, ld: int, dist: str, seed: int, dtype=torch.float64, poison=float("nan"),
           device="cpu", chunk_cols: int | None = None) -> torch.Tensor:
    """Flat column-major storage (``ld*cols`` elements) of a rows x cols matrix drawn from ``dist``.

    Element (r, c) depends only on (seed, r + c*rows): the leading dimension does not change the
    values.  fp32 data are the fp64 draws rounded to nearest.  complex128 draws real and imaginary
    parts from seeds ``seed`` and ``seed + 1``.
    """
    if ld < max(1, rows):
        raise ValueError("ld must be at least max(1, rows)")
    if dtype == torch.complex128:
        re = matrix(rows, cols, ld, dist, seed, torch.float64, poison, device, chunk_cols)
        im = matrix(rows, cols, ld, dist, seed + 1, torch.float64, poison, device, chunk_cols)
        return torch.complex(re, im)
    out = torch.full((max(cols, 0) * ld,), poison, dtype=dtype, device=device)
    if rows == 0 or cols == 0:
        return out
    view = out.view(cols, ld)
    step = chunk_cols or max(1, (1 << 24) // max(rows, 1))
    r = torch.arange(rows, dtype=torch.int64, device=device)
    for c0 in range(0, cols, step):
        c1 = min(cols, c0 + step)
        idx = r.unsqueeze(0) + torch.arange(c0, c1, dtype=torch.int64, device=device).unsqueeze(1) * rows
        view[c0:c1, :rows] = _values(dist, seed, idx).to(dtype)
    return out


def operand_shapes(transa: str, transb: str, m: int, n: int, k: int):
    """(rows, cols) of the stored A and B for the given transposes."""
    a = (m, k) if transa in "Nn" else (k, m)
    b = (k, n) if transb in "Nn" else (n, k)
    return a, b


def padded_ld(rows: int) -> int:
    """Leading dimension 'next multiple of 32, plus 3' used by the fringe/transposition workload."""
    return ((max(rows, 1) + 31) // 32) * 32 + 3


def gemm_inputs(transa, transb, m, n, k, dist, seed, dtype=torch.float64, lda=None, ldb=None, ldc=None, device="cpu",
                c_dist=None):
    """A, B, C storage for one GEMM problem (seeds ``seed``, ``seed+101``, ``seed+202``) and their leading dimensions.

    ``c_dist`` = "zero" gives a zero C; default draws C from ``dist``.
    """
    (ra, ca), (rb, cb) = operand_shapes(transa, transb, m, n, k)
    lda = max(1, ra) if lda is None else lda
    ldb = max(1, rb) if ldb is None else ldb
    ldc = max(1, m) if ldc is None else ldc
    A = matrix(ra, ca, lda, dist, seed, dtype, float("nan"), device)
    B = matrix(rb, cb, ldb, dist, seed + 101, dtype, float("nan"), device)
    if c_dist == "zero":
        C = torch.full((max(n, 0) * ldc,), C_SENTINEL, dtype=dtype, device=device)
        if m and n:
            C.view(n, ldc)[:, :m] = 0
    else:
        C = matrix(m, n, ldc, c_dist or dist, seed + 202, dtype, C_SENTINEL, device)
    return A, lda, B, ldb, C, ldc
