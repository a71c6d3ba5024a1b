"""Test-side helpers: BLAS storage from 2-D arrays, error-bound checks.  No GEMM arithmetic of the product."""
from __future__ import annotations

import numpy as np

U = {np.dtype(np.float64): 2.0 ** -53, np.dtype(np.float32): 2.0 ** -24, np.dtype(np.complex128): 2.0 ** -53}
SENTINEL = -7.25e11


def store(X: np.ndarray, ld: int, poison) -> np.ndarray:
    """Flat column-major storage with leading dimension ld of the 2-D array X; padding rows = poison."""
    rows, cols = X.shape
    assert ld >= max(1, rows)
    out = np.full(ld * cols, poison, dtype=X.dtype)
    if rows and cols:
        out.reshape(cols, ld)[:, :rows] = X.T
    return out


def unstore(flat: np.ndarray, rows: int, cols: int, ld: int) -> np.ndarray:
    """The rows x cols matrix held in flat column-major storage."""
    if rows == 0 or cols == 0:
        return np.zeros((rows, cols), dtype=flat.dtype)
    return flat[: ld * cols].reshape(cols, ld)[:, :rows].T.copy()


def padding(flat: np.ndarray, rows: int, cols: int, ld: int) -> np.ndarray:
    return flat[: ld * cols].reshape(cols, ld)[:, rows:].copy()


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    """Bitwise equality (NaN == NaN, +0 != -0)."""
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.shape == b.shape and a.dtype == b.dtype and a.tobytes() == b.tobytes()
