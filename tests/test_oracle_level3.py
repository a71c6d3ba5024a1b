"""Pins of the level-3 oracles: SYRK against the GEMM oracle on the same operand (bitwise on the triangle), exact
rational brute force, symmetry, integer closed form, the untouched triangle; strided-batched GEMM against
per-problem calls."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from helpers import SENTINEL, bits_equal, store, unstore


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_syrk_equals_gemm_triangle_and_leaves_the_rest(oracle, dtype):
    rng = np.random.default_rng(1)
    n, k = 23, 17
    for uplo, trans in itertools.product("LU", "NT"):
        ra, ca = (n, k) if trans == "N" else (k, n)
        A2 = rng.uniform(-1, 1, (ra, ca)).astype(dtype)
        C2 = rng.uniform(-1, 1, (n, n)).astype(dtype)
        A = store(A2, ra + 2, np.nan)
        C = store(C2, n + 3, SENTINEL)
        oracle.ref_syrk(uplo, trans, n, k, 0.7, A, ra + 2, -0.3, C, n + 3)
        G = store(C2, n + 3, SENTINEL)
        oracle.ref_gemm(trans, "T" if trans == "N" else "N", n, n, k, 0.7, A, ra + 2, A, ra + 2, -0.3, G, n + 3)
        got, full = unstore(C, n, n, n + 3), unstore(G, n, n, n + 3)
        tri = np.tril(np.ones((n, n), bool)) if uplo == "L" else np.triu(np.ones((n, n), bool))
        assert bits_equal(got[tri], full[tri])
        assert bits_equal(got[~tri], C2[~tri])  # the other triangle is not touched
        assert bits_equal(C.reshape(n, n + 3)[:, n:], np.full((n, 3), SENTINEL, dtype))


def test_syrk_rational_brute_force_and_symmetry(oracle):
    rng = np.random.default_rng(2)
    for n, k in itertools.product([0, 1, 2, 3, 5], [0, 1, 2, 4]):
        for trans in "NT":
            ra, ca = (n, k) if trans == "N" else (k, n)
            A2 = (rng.integers(-16, 17, (ra, ca)) / 8.0)
            C2 = (rng.integers(-16, 17, (n, n)) / 8.0)
            out = {}
            for uplo in "LU":
                C = store(C2, max(1, n), SENTINEL)
                oracle.ref_syrk(uplo, trans, n, k, -1.0, store(A2, max(1, ra), np.nan), max(1, ra), 0.5, C, max(1, n))
                out[uplo] = unstore(C, n, n, max(1, n))
            opA = A2 if trans == "N" else A2.T
            for i in range(n):
                for j in range(n):
                    want = -sum(Fraction(float(opA[i, p])) * Fraction(float(opA[j, p])) for p in range(k)) \
                           + Fraction(0.5) * Fraction(float(C2[i, j]))
                    got = out["L"][i, j] if i >= j else out["U"][i, j]
                    assert Fraction(float(got)) == want
    # the two triangles of A A^T computed separately are transposes of each other bit for bit
    n, k = 19, 33
    A2 = rng.uniform(-1, 1, (n, k))
    L, U = np.zeros(n * n), np.zeros(n * n)
    oracle.ref_syrk("L", "N", n, k, 1.0, store(A2, n, np.nan), n, 0.0, L, n)
    oracle.ref_syrk("U", "N", n, k, 1.0, store(A2, n, np.nan), n, 0.0, U, n)
    assert bits_equal(np.tril(unstore(L, n, n, n)), np.triu(unstore(U, n, n, n)).T)


def test_syrk_quick_returns_and_errors(oracle):
    n, k = 6, 4
    rng = np.random.default_rng(3)
    C2 = rng.uniform(-1, 1, (n, n))
    nanA = np.full(n * k, np.nan)
    C = store(C2, n, SENTINEL)
    oracle.ref_syrk("L", "N", n, k, 0.0, nanA, n, 0.5, C, n)
    got = unstore(C, n, n, n)
    assert bits_equal(np.tril(got), np.tril(0.5 * C2)) and bits_equal(np.triu(got, 1), np.triu(C2, 1))
    C = store(np.full((n, n), np.nan), n, SENTINEL)
    oracle.ref_syrk("U", "T", n, k, 1.0, store(rng.uniform(-1, 1, (k, n)), k, np.nan), k, 0.0, C, n)
    got = unstore(C, n, n, n)
    assert np.all(np.isfinite(got[np.triu_indices(n)])) and np.all(np.isnan(got[np.tril_indices(n, -1)]))
    z = np.zeros(64)
    for args, idx in [(("X", "N", 2, 2, 1.0, z, 2, 0.0, z, 2), 1), (("L", "Q", 2, 2, 1.0, z, 2, 0.0, z, 2), 2),
                      (("L", "N", -1, 2, 1.0, z, 2, 0.0, z, 2), 3), (("L", "N", 2, -1, 1.0, z, 2, 0.0, z, 2), 4),
                      (("L", "N", 3, 2, 1.0, z, 2, 0.0, z, 3), 7), (("L", "T", 3, 4, 1.0, z, 3, 0.0, z, 3), 7),
                      (("L", "N", 3, 2, 1.0, z, 3, 0.0, z, 2), 10)]:
        with pytest.raises(ValueError, match=f"argument {idx}$"):
            oracle.ref_syrk(*args)


def test_strided_batched_is_per_problem_gemm(oracle):
    rng = np.random.default_rng(4)
    m, n, k, batch = 5, 4, 7, 3
    sa, sb, sc = m * k + 3, 0, (m + 1) * n + 2  # B shared by all problems
    A = rng.uniform(-1, 1, sa * batch)
    B = rng.uniform(-1, 1, k * n)
    C0 = rng.uniform(-1, 1, sc * batch)
    C = C0.copy()
    oracle.ref_gemm_strided_batched("N", "N", m, n, k, 0.7, A, m, sa, B, k, sb, -0.3, C, m + 1, sc, batch)
    for b in range(batch):
        want = 0.7 * (A[b * sa:b * sa + m * k].reshape(k, m).T @ B.reshape(n, k).T) \
               - 0.3 * C0[b * sc:b * sc + (m + 1) * n].reshape(n, m + 1)[:, :m].T
        got = C[b * sc:b * sc + (m + 1) * n].reshape(n, m + 1)[:, :m].T
        assert np.allclose(got, want, rtol=0, atol=1e-14)
        gap = C[b * sc + (m + 1) * n:(b + 1) * sc]
        assert bits_equal(gap, C0[b * sc + (m + 1) * n:(b + 1) * sc])
