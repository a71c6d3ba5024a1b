"""Pins of the triangular level-3 oracles (TRMM, TRSM).

TRMM: bit for bit the GEMM oracle applied to the explicitly zero-filled triangular matrix (adding exact zeros
changes nothing), numpy on exact integer data.  TRSM: scipy's solve_triangular (an independent library routine),
exact integer systems against Python-integer substitution, diagonal systems in closed form, the componentwise
residual bound of substitution, and TRSM undoing TRMM.  Both: only the named triangle is read, a unit diagonal
is not read, quick returns, argument errors."""
import itertools

import numpy as np
import pytest
import scipy.linalg

from helpers import SENTINEL, bits_equal, store, unstore

COMBOS = list(itertools.product("LR", "LU", "NT", "NU"))


def tri_matrix(rng, na, uplo, diag, dtype, well_conditioned=True):
    """Dense na x na array whose `uplo` triangle holds the matrix and whose other triangle is NaN; with diag 'U'
    the diagonal is NaN too (it must not be read).  Returns (stored, logical)."""
    off = rng.uniform(-1, 1, (na, na)) / (max(na, 1) if well_conditioned else 1)
    d = rng.uniform(1, 2, na) * rng.choice([-1, 1], na)
    logical = (np.tril(off, -1) if uplo == "L" else np.triu(off, 1)) + np.diag(np.ones(na) if diag == "U" else d)
    logical = logical.astype(dtype)
    stored = logical.copy()
    mask = np.triu(np.ones((na, na), bool), 1) if uplo == "L" else np.tril(np.ones((na, na), bool), -1)
    stored[mask] = np.nan
    if diag == "U":
        stored[np.diag_indices(na)] = np.nan
    return stored, logical


def op(T, trans):
    return T if trans == "N" else T.T


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_trmm_equals_gemm_with_the_dense_triangle(oracle, dtype):
    rng = np.random.default_rng(31)
    m, n = 19, 13
    for side, uplo, trans, diag in COMBOS:
        na = m if side == "L" else n
        stored, logical = tri_matrix(rng, na, uplo, diag, dtype)
        B2 = rng.uniform(-1, 1, (m, n)).astype(dtype)
        A = store(stored, na + 2, np.nan)
        B = store(B2, m + 3, SENTINEL)
        oracle.ref_trmm(side, uplo, trans, diag, m, n, 0.7, A, na + 2, B, m + 3)
        dense = store(logical, na, np.nan)
        C = store(np.zeros((m, n), dtype), m, SENTINEL)
        Bd = store(B2, m, np.nan)
        if side == "L":
            oracle.ref_gemm(trans, "N", m, n, m, 0.7, dense, na, Bd, m, 0.0, C, m)
        else:
            oracle.ref_gemm("N", trans, m, n, n, 0.7, Bd, m, dense, na, 0.0, C, m)
        assert bits_equal(unstore(B, m, n, m + 3), unstore(C, m, n, m)), (side, uplo, trans, diag)
        assert bits_equal(B.reshape(n, m + 3)[:, m:], np.full((n, 3), SENTINEL, dtype))


def test_trmm_and_trsm_exact_on_integers(oracle):
    """Unit-diagonal triangular matrices with entries in {-1, 0, 1} on two off-diagonals and integer right-hand
    sides: products and solutions are integers of moderate size, so there is one correct bit pattern; it is
    computed here with Python integers."""
    rng = np.random.default_rng(32)
    m, n = 24, 9
    for side, uplo, trans, diag in COMBOS:
        na = m if side == "L" else n
        band = np.zeros((na, na), dtype=np.int64)
        for o in (1, 2):
            vals = rng.integers(-1, 2, na - o)
            band += np.diag(vals, -o if uplo == "L" else o)
        dvals = np.ones(na, dtype=np.int64) if diag == "U" else rng.choice([-1, 1, 2, -2], na)
        logical = band + np.diag(dvals)
        stored = logical.astype(np.float64)
        if diag == "U":
            stored[np.diag_indices(na)] = np.nan
        T = op(logical, trans).astype(object)
        X2 = rng.integers(-3, 4, (m, n)).astype(object)
        prod = (T.dot(X2) if side == "L" else X2.dot(T))
        A = store(stored, na, np.nan)
        # TRMM: B := 2 * T * X
        B = store(X2.astype(np.float64), m, SENTINEL)
        oracle.ref_trmm(side, uplo, trans, diag, m, n, 2.0, A, na, B, m)
        assert np.array_equal(unstore(B, m, n, m), (2 * prod).astype(np.float64))
        # TRSM: solve T * Y = 0.5 * (2 * T * X)  ->  Y = X exactly (powers of two in the diagonal and alpha)
        oracle.ref_trsm(side, uplo, trans, diag, m, n, 0.5, A, na, B, m)
        assert np.array_equal(unstore(B, m, n, m), X2.astype(np.float64)), (side, uplo, trans, diag)


@pytest.mark.parametrize("dtype,tol", [(np.float64, 1e-13), (np.float32, 5e-5)])
def test_trsm_against_scipy_and_residual_bound(oracle, dtype, tol):
    rng = np.random.default_rng(33)
    m, n = 41, 17
    u = 2.0 ** -53 if dtype == np.float64 else 2.0 ** -24
    for side, uplo, trans, diag in COMBOS:
        na = m if side == "L" else n
        stored, logical = tri_matrix(rng, na, uplo, diag, dtype)
        B2 = rng.uniform(-1, 1, (m, n)).astype(dtype)
        alpha = 0.7
        B = store(B2, m + 1, SENTINEL)
        oracle.ref_trsm(side, uplo, trans, diag, m, n, alpha, store(stored, na + 1, np.nan), na + 1, B, m + 1)
        X = unstore(B, m, n, m + 1).astype(np.float64)
        T = op(logical.astype(np.float64), trans)
        rhs = float(dtype(alpha)) * B2.astype(np.float64)
        if side == "L":
            want = scipy.linalg.solve_triangular(T, rhs, lower=(uplo == "L") != (trans == "T"))
            resid, mag = T @ X - rhs, np.abs(T) @ np.abs(X) + np.abs(rhs)
        else:
            want = scipy.linalg.solve_triangular(T.T, rhs.T, lower=(uplo == "L") == (trans == "T")).T
            resid, mag = X @ T - rhs, np.abs(X) @ np.abs(T) + np.abs(rhs)
        assert np.allclose(X, want, rtol=tol, atol=tol), (side, uplo, trans, diag)
        assert np.all(np.abs(resid) <= (na + 3) * u * mag), (side, uplo, trans, diag)
        assert bits_equal(B.reshape(n, m + 1)[:, m:], np.full((n, 1), SENTINEL, dtype))


def test_trsm_diagonal_and_identity_closed_forms(oracle):
    rng = np.random.default_rng(34)
    m, n = 7, 5
    d = rng.uniform(1, 2, m)
    B2 = rng.uniform(-1, 1, (m, n))
    A = store(np.diag(d), m, np.nan)
    for uplo, trans in itertools.product("LU", "NT"):
        B = store(B2, m, SENTINEL)
        oracle.ref_trsm("L", uplo, trans, "N", m, n, 0.3, A, m, B, m)
        assert bits_equal(unstore(B, m, n, m), (0.3 * B2 - 0.0) / d[:, None])  # two roundings: alpha*b, then / d
        B = store(B2, m, SENTINEL)
        oracle.ref_trsm("L", uplo, trans, "U", m, n, 0.3, A, m, B, m)  # unit diagonal: A's diagonal is ignored
        assert bits_equal(unstore(B, m, n, m), 0.3 * B2 - 0.0)


def test_trsm_undoes_trmm(oracle):
    rng = np.random.default_rng(35)
    m, n = 33, 21
    for side, uplo, trans, diag in COMBOS:
        na = m if side == "L" else n
        stored, _ = tri_matrix(rng, na, uplo, diag, np.float64)
        A = store(stored, na, np.nan)
        X2 = rng.uniform(-1, 1, (m, n))
        B = store(X2, m, SENTINEL)
        oracle.ref_trmm(side, uplo, trans, diag, m, n, 1.0, A, na, B, m)
        oracle.ref_trsm(side, uplo, trans, diag, m, n, 1.0, A, na, B, m)
        assert np.allclose(unstore(B, m, n, m), X2, rtol=0, atol=1e-13)


def test_triangular_quick_returns_and_errors(oracle):
    nanA = np.full(16, np.nan)
    for fn in (oracle.ref_trmm, oracle.ref_trsm):
        B = store(np.ones((4, 3)), 5, SENTINEL)
        fn("L", "L", "N", "N", 4, 3, 0.0, nanA, 4, B, 5)  # alpha == 0: zeros, A is not read
        assert np.array_equal(unstore(B, 4, 3, 5), np.zeros((4, 3)))
        assert np.all(B.reshape(3, 5)[:, 4:] == SENTINEL)
        fn("R", "U", "T", "U", 0, 3, 1.0, nanA, 3, B, 1)
        fn("L", "U", "T", "U", 4, 0, 1.0, nanA, 4, B, 4)
        for bad in (("X", "L", "N", "N", 4, 3, 4, 5), ("L", "X", "N", "N", 4, 3, 4, 5), ("L", "L", "X", "N", 4, 3, 4, 5),
                    ("L", "L", "N", "X", 4, 3, 4, 5), ("L", "L", "N", "N", -1, 3, 4, 5), ("L", "L", "N", "N", 4, -1, 4, 5),
                    ("L", "L", "N", "N", 4, 3, 3, 5), ("R", "L", "N", "N", 4, 3, 2, 5), ("L", "L", "N", "N", 4, 3, 4, 3)):
            side, uplo, trans, diag, m, n, lda, ldb = bad
            with pytest.raises(ValueError):
                fn(side, uplo, trans, diag, m, n, 1.0, nanA, lda, B, ldb)
