"""Pins of the CPU oracle against things other than itself.

The paper prints no numeric GEMM example (its figures are symbolic register layouts), so the
oracle is pinned by: exact rational brute force on tiny shapes, identity/zero matrices, the
transpose identity (AB)^T = B^T A^T, integer-valued inputs evaluated in int64, textbook
special cases (rank-1 update, dot product), the standard inner-product error bound between
the working-precision and wide oracles, and 4M complex against direct complex arithmetic.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from helpers import SENTINEL, U, bits_equal, padding, store, unstore

TRANS = list(itertools.product("NT", "NT"))


def op_shapes(ta, tb, m, n, k):
    return ((m, k) if ta == "N" else (k, m)), ((k, n) if tb == "N" else (n, k))


def dyadic(rng, shape, dtype=np.float64):
    """Multiples of 1/8 in [-2, 2]: every product and short sum is exact in fp32 and fp64."""
    return (rng.integers(-16, 17, size=shape) / 8.0).astype(dtype)


def exact_gemm(ta, tb, m, n, k, alpha, A2, B2, beta, C2):
    """Independent evaluation in exact rational arithmetic from the 2-D stored operands."""
    opA = A2 if ta == "N" else A2.T
    opB = B2 if tb == "N" else B2.T
    out = [[None] * n for _ in range(m)]
    for i in range(m):
        for j in range(n):
            s = Fraction(0)
            for p in range(k):
                s += Fraction(float(opA[i, p])) * Fraction(float(opB[p, j]))
            out[i][j] = Fraction(float(alpha)) * s + Fraction(float(beta)) * Fraction(float(C2[i, j]))
    return out


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_brute_force_tiny_shapes_exact(oracle, dtype):
    """All m, n, k in {0,1,2,3,5}, four transposes, two leading dimensions, alpha/beta in {0,1,-1,0.5}:
    on dyadic inputs every operation is exact, so the oracle must equal the rational result."""
    rng = np.random.default_rng(11)
    sizes = [0, 1, 2, 3, 5]
    scal = [0.0, 1.0, -1.0, 0.5]
    count = 0
    for (ta, tb), m, n, k in itertools.product(TRANS, sizes, sizes, sizes):
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        A2, B2, C2 = dyadic(rng, (ra, ca), dtype), dyadic(rng, (rb, cb), dtype), dyadic(rng, (m, n), dtype)
        for extra in (0, 3):
            lda, ldb, ldc = max(1, ra) + extra, max(1, rb) + extra, max(1, m) + extra
            alpha, beta = scal[count % 4], scal[(count // 4) % 4]
            count += 1
            A, B = store(A2, lda, np.nan), store(B2, ldb, np.nan)
            C = store(C2, ldc, SENTINEL)
            oracle.ref_gemm(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc)
            want = exact_gemm(ta, tb, m, n, k, alpha, A2, B2, beta, C2)
            got = unstore(C, m, n, ldc)
            for i in range(m):
                for j in range(n):
                    assert Fraction(float(got[i, j])) == want[i][j], (ta, tb, m, n, k, alpha, beta, i, j)
            assert np.all(padding(C, m, n, ldc) == SENTINEL)
    assert count == 4 * 125 * 2


@pytest.mark.parametrize("alpha,beta", list(itertools.product([0.0, 1.0, -1.0, 0.5], repeat=2)))
def test_every_alpha_beta_pair_exact(oracle, alpha, beta):
    rng = np.random.default_rng(5)
    for ta, tb in TRANS:
        m, n, k = 4, 3, 5
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        A2, B2, C2 = dyadic(rng, (ra, ca)), dyadic(rng, (rb, cb)), dyadic(rng, (m, n))
        A, B, C = store(A2, ra + 3, np.nan), store(B2, rb + 3, np.nan), store(C2, m + 3, SENTINEL)
        oracle.ref_gemm(ta, tb, m, n, k, alpha, A, ra + 3, B, rb + 3, beta, C, m + 3)
        want = exact_gemm(ta, tb, m, n, k, alpha, A2, B2, beta, C2)
        got = unstore(C, m, n, m + 3)
        assert all(Fraction(float(got[i, j])) == want[i][j] for i in range(m) for j in range(n))


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_random_inputs_within_inner_product_bound_of_exact(oracle, dtype):
    """On general inputs the oracle (and the wide oracle) stay within (k+2)*u*S of the exact value, and the
    magnitude sum S the wide oracle returns equals the exact one to rounding."""
    rng = np.random.default_rng(3)
    u = U[np.dtype(dtype)]
    for ta, tb in TRANS:
        m, n, k = 5, 4, 23
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        A2 = rng.uniform(-1, 1, (ra, ca)).astype(dtype)
        B2 = rng.uniform(-1, 1, (rb, cb)).astype(dtype)
        C2 = rng.uniform(-1, 1, (m, n)).astype(dtype)
        alpha, beta = dtype(0.7), dtype(-0.3)
        A, B, C = store(A2, ra + 1, np.nan), store(B2, rb + 2, np.nan), store(C2, m + 3, SENTINEL)
        Chi, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A, ra + 1, B, rb + 2, beta, C, m + 3)
        oracle.ref_gemm(ta, tb, m, n, k, alpha, A, ra + 1, B, rb + 2, beta, C, m + 3)
        got, hi, S2 = unstore(C, m, n, m + 3), unstore(Chi, m, n, m), unstore(S, m, n, m)
        want = exact_gemm(ta, tb, m, n, k, alpha, A2, B2, beta, C2)
        opA = A2 if ta == "N" else A2.T
        opB = B2 if tb == "N" else B2.T
        for i in range(m):
            for j in range(n):
                s_exact = abs(Fraction(float(alpha))) * sum(
                    abs(Fraction(float(opA[i, p])) * Fraction(float(opB[p, j]))) for p in range(k)) + abs(
                        Fraction(float(beta)) * Fraction(float(C2[i, j])))
                assert abs(float(S2[i, j]) - float(s_exact)) <= 1e-12 * float(s_exact)
                assert abs(Fraction(float(got[i, j])) - want[i][j]) <= (k + 2) * u * s_exact
                assert abs(Fraction(float(hi[i, j])) - want[i][j]) <= 1.01 * u * s_exact  # one final rounding


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_identity_and_zero_matrices(oracle, dtype):
    rng = np.random.default_rng(1)
    n = 17
    B2 = rng.uniform(-1, 1, (n, n)).astype(dtype)
    C2 = rng.uniform(-1, 1, (n, n)).astype(dtype)
    alpha, beta = dtype(1.5), dtype(0.5)
    eye = np.eye(n, dtype=dtype)
    for ta, tb in TRANS:
        # A = I: every sum has exactly one non-zero term, so C = alpha*op(B) + beta*C with the oracle's roundings
        C = store(C2, n, SENTINEL)
        oracle.ref_gemm(ta, tb, n, n, n, alpha, store(eye, n, np.nan), n, store(B2, n, np.nan), n, beta, C, n)
        opB = B2 if tb == "N" else B2.T
        assert bits_equal(unstore(C, n, n, n), (alpha * opB + beta * C2).astype(dtype))
        # B = I
        C = store(C2, n, SENTINEL)
        oracle.ref_gemm(ta, tb, n, n, n, alpha, store(B2, n, np.nan), n, store(eye, n, np.nan), n, beta, C, n)
        opA = B2 if ta == "N" else B2.T
        assert bits_equal(unstore(C, n, n, n), (alpha * opA + beta * C2).astype(dtype))
        # A = 0: C = alpha*0 + beta*C
        C = store(C2, n, SENTINEL)
        oracle.ref_gemm(ta, tb, n, n, n, alpha, store(np.zeros((n, n), dtype), n, np.nan), n, store(B2, n, np.nan), n,
                        beta, C, n)
        assert bits_equal(unstore(C, n, n, n), (beta * C2).astype(dtype) + dtype(0))


def test_quick_return_rules_and_nan_poison(oracle):
    rng = np.random.default_rng(2)
    m, n, k = 6, 5, 4
    A2, B2, C2 = rng.uniform(-1, 1, (m, k)), rng.uniform(-1, 1, (k, n)), rng.uniform(-1, 1, (m, n))
    nanA, nanB, nanC = np.full((m, k), np.nan), np.full((k, n), np.nan), np.full((m, n), np.nan)
    # beta == 0: the old C (NaN) must not propagate
    C = store(nanC, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, 1.0, store(A2, m, np.nan), m, store(B2, k, np.nan), k, 0.0, C, m)
    assert np.all(np.isfinite(unstore(C, m, n, m)))
    # alpha == 0: A and B (NaN) are not referenced; C = beta*C
    C = store(C2, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, 0.0, store(nanA, m, np.nan), m, store(nanB, k, np.nan), k, 0.5, C, m)
    assert bits_equal(unstore(C, m, n, m), 0.5 * C2)
    # alpha == 0 and beta == 0: zeros
    C = store(nanC, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, 0.0, store(nanA, m, np.nan), m, store(nanB, k, np.nan), k, 0.0, C, m)
    assert np.all(unstore(C, m, n, m) == 0.0)
    # k == 0: C = beta*C
    C = store(C2, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, 0, 1.0, np.zeros(0), m, np.zeros(0), 1, -1.0, C, m)
    assert bits_equal(unstore(C, m, n, m), -C2)
    # alpha == 0, beta == 1 and m == 0 / n == 0: nothing is touched
    C = store(C2, m, SENTINEL)
    before = C.copy()
    oracle.ref_gemm("N", "N", m, n, k, 0.0, store(nanA, m, np.nan), m, store(nanB, k, np.nan), k, 1.0, C, m)
    oracle.ref_gemm("N", "N", 0, n, k, 1.0, np.zeros(0), 1, store(B2, k, np.nan), k, 0.0, C, m)
    oracle.ref_gemm("N", "N", m, 0, k, 1.0, store(A2, m, np.nan), m, np.zeros(0), k, 0.0, C, m)
    assert bits_equal(C, before)
    # NaN in A propagates when alpha != 0 (no shortcut on zero B)
    A3 = A2.copy()
    A3[2, 1] = np.nan
    C = store(np.zeros((m, n)), m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, 1.0, store(A3, m, np.nan), m, store(np.zeros((k, n)), k, np.nan), k, 0.0, C, m)
    got = unstore(C, m, n, m)
    assert np.all(np.isnan(got[2, :])) and np.all(got[[0, 1, 3, 4, 5], :] == 0.0)


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_transpose_identity_bitwise(oracle, dtype):
    """(AB)^T = B^T A^T: gemm(N,N,m,n,k,A,B) and gemm(T,T,n,m,k,B,A) on the same stored arrays give transposed
    results bit for bit (same products, same ascending-p order; multiplication commutes).  Likewise N/T and T/N
    against explicitly transposed copies."""
    rng = np.random.default_rng(4)
    m, n, k = 13, 9, 31
    A2 = rng.uniform(-1, 1, (m, k)).astype(dtype)
    B2 = rng.uniform(-1, 1, (k, n)).astype(dtype)
    alpha = dtype(0.7)
    X = np.zeros(m * n, dtype)
    oracle.ref_gemm("N", "N", m, n, k, alpha, store(A2, m, np.nan), m, store(B2, k, np.nan), k, 0.0, X, m)
    Y = np.zeros(n * m, dtype)
    oracle.ref_gemm("T", "T", n, m, k, alpha, store(B2, k, np.nan), k, store(A2, m, np.nan), m, 0.0, Y, n)
    assert bits_equal(unstore(X, m, n, m), unstore(Y, n, m, n).T)
    # explicit transposes: op(A^T stored) with T equals op(A stored) with N
    for ta, tb in TRANS:
        As = A2 if ta == "N" else np.ascontiguousarray(A2.T)
        Bs = B2 if tb == "N" else np.ascontiguousarray(B2.T)
        Z = np.zeros(m * n, dtype)
        oracle.ref_gemm(ta, tb, m, n, k, alpha, store(As, As.shape[0] + 2, np.nan), As.shape[0] + 2,
                        store(Bs, Bs.shape[0] + 1, np.nan), Bs.shape[0] + 1, 0.0, Z, m)
        assert bits_equal(Z, X), (ta, tb)


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_integer_inputs_match_int64_closed_form(oracle, dtype):
    """Entries in {-4..4}, alpha = 1.5, beta = 0.5: 2*C_new = 3*acc + C_old in exact integer arithmetic."""
    rng = np.random.default_rng(6)
    for ta, tb in TRANS:
        m, n, k = 37, 29, 301
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        Ai, Bi, Ci = (rng.integers(-4, 5, s) for s in ((ra, ca), (rb, cb), (m, n)))
        C = store(Ci.astype(dtype), m + 3, SENTINEL)
        oracle.ref_gemm(ta, tb, m, n, k, 1.5, store(Ai.astype(dtype), ra, np.nan), ra, store(Bi.astype(dtype), rb, np.nan),
                        rb, 0.5, C, m + 3)
        acc = (Ai if ta == "N" else Ai.T).astype(np.int64) @ (Bi if tb == "N" else Bi.T).astype(np.int64)
        twice = 3 * acc + Ci
        got = unstore(C, m, n, m + 3).astype(np.float64)
        assert np.array_equal(got * 2.0, twice.astype(np.float64))


def test_rank1_dot_and_slice_special_cases(oracle):
    rng = np.random.default_rng(7)
    m, n = 11, 7
    a, b, C2 = rng.uniform(-1, 1, (m, 1)), rng.uniform(-1, 1, (1, n)), rng.uniform(-1, 1, (m, n))
    alpha, beta = 0.7, -0.3
    # k = 1: rank-1 update, each element is fl(fl(alpha*fl(a_i*b_j)) + fl(beta*c_ij))
    C = store(C2, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, 1, alpha, store(a, m, np.nan), m, store(b, 1, np.nan), 1, beta, C, m)
    assert bits_equal(unstore(C, m, n, m), alpha * (a * b) + beta * C2)
    # m = n = 1: a dot product; compare with the correctly rounded sum (math.fsum of exact products is not
    # available in floats, so use rationals) within the k*u bound
    k = 257
    x, y = rng.uniform(-1, 1, k), rng.uniform(-1, 1, k)
    C = np.zeros(1)
    oracle.ref_gemm("T", "N", 1, 1, k, 1.0, x.copy(), k, y.copy(), k, 0.0, C, 1)
    exact = sum(Fraction(float(p)) * Fraction(float(q)) for p, q in zip(x, y))
    mag = sum(abs(Fraction(float(p)) * Fraction(float(q))) for p, q in zip(x, y))
    assert abs(Fraction(float(C[0])) - exact) <= k * 2.0 ** -53 * mag
    # column j of C depends only on column j of op(B): a column subset equals the same columns of the full run
    k = 19
    A2, B2 = rng.uniform(-1, 1, (m, k)), rng.uniform(-1, 1, (k, n))
    full = store(C2, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, alpha, store(A2, m, np.nan), m, store(B2, k, np.nan), k, beta, full, m)
    part = store(C2, m, SENTINEL)
    cols = [5, 0, 3]
    oracle.ref_gemm("N", "N", m, n, k, alpha, store(A2, m, np.nan), m, store(B2, k, np.nan), k, beta, part, m, cols=cols)
    f2, p2 = unstore(full, m, n, m), unstore(part, m, n, m)
    assert bits_equal(p2[:, cols], f2[:, cols])
    rest = [j for j in range(n) if j not in cols]
    assert bits_equal(p2[:, rest], C2[:, rest])


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_working_vs_wide_oracle_bound(oracle, dtype):
    """|ref - ref_hi| <= (k+2)*u*S elementwise (standard inner-product bound) on a mid-sized problem."""
    rng = np.random.default_rng(8)
    u = U[np.dtype(dtype)]
    m, n, k = 96, 80, 513
    for ta, tb in TRANS:
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        A = store(rng.uniform(-1, 1, (ra, ca)).astype(dtype), ra + 3, np.nan)
        B = store(rng.uniform(-1, 1, (rb, cb)).astype(dtype), rb + 3, np.nan)
        C = store(rng.uniform(-1, 1, (m, n)).astype(dtype), m + 3, SENTINEL)
        hi, S = oracle.ref_gemm_hi(ta, tb, m, n, k, 0.7, A, ra + 3, B, rb + 3, -0.3, C, m + 3)
        oracle.ref_gemm(ta, tb, m, n, k, 0.7, A, ra + 3, B, rb + 3, -0.3, C, m + 3)
        diff = np.abs(unstore(C, m, n, m + 3).astype(np.float64) - unstore(hi, m, n, m).astype(np.float64))
        assert np.all(diff <= (k + 2) * u * unstore(S, m, n, m))
        assert diff.max() > 0  # the two really accumulate differently


def test_fp32_oracle_accumulates_in_fp32(oracle):
    """The fp32 oracle rounds every product and every partial sum to fp32 (it is not a double accumulation):
    on a case where fp32 accumulation visibly loses bits, it differs from the wide result but equals a
    step-by-step fp32 evaluation."""
    k = 1000
    x = np.full(k, np.float32(0.1))
    y = np.full(k, np.float32(0.3))
    C = np.zeros(1, np.float32)
    oracle.ref_gemm("T", "N", 1, 1, k, 1.0, x, k, y, k, 0.0, C, 1)
    acc = np.float32(0)
    for p in range(k):
        acc = np.float32(acc + np.float32(x[p] * y[p]))
    assert C[0] == acc
    hi, _ = oracle.ref_gemm_hi("T", "N", 1, 1, k, 1.0, x, k, y, k, 0.0, np.zeros(1, np.float32), 1)
    assert hi[0] != C[0]


def test_complex_direct_vs_4m(oracle):
    """4M on split planes against direct complex arithmetic: bitwise on integer-valued inputs (both exact),
    within the complex bound on general inputs; and direct complex against numpy on a tiny exact case."""
    rng = np.random.default_rng(9)
    m, n, k = 9, 7, 12
    for ta, tb in TRANS:
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)

        def zint(shape):
            return (rng.integers(-4, 5, shape) + 1j * rng.integers(-4, 5, shape)).astype(np.complex128)

        A2, B2, C2 = zint((ra, ca)), zint((rb, cb)), zint((m, n))
        for alpha, beta in (((1 + 0.5j), 0j), ((2 - 1j), (0.5 + 0.5j)), (1 + 0j, 1 + 0j)):
            Cd = store(C2, m + 1, SENTINEL)
            C4 = store(C2, m + 1, SENTINEL)
            A, B = store(A2, ra + 2, np.nan), store(B2, rb + 2, np.nan)
            oracle.ref_gemm(ta, tb, m, n, k, alpha, A, ra + 2, B, rb + 2, beta, Cd, m + 1)
            oracle.ref_zgemm_4m(ta, tb, m, n, k, alpha, A, ra + 2, B, rb + 2, beta, C4, m + 1)
            assert bits_equal(unstore(Cd, m, n, m + 1), unstore(C4, m, n, m + 1))
            want = alpha * ((A2 if ta == "N" else A2.T) @ (B2 if tb == "N" else B2.T)) + beta * C2
            assert np.array_equal(unstore(Cd, m, n, m + 1), want)  # exact in integers
            assert np.all(padding(Cd, m, n, m + 1).real == SENTINEL)
    # general inputs: within 2*(2k+4)*u*S of each other and of the wide result
    m, n, k = 24, 20, 65
    A2 = rng.uniform(-1, 1, (m, k)) + 1j * rng.uniform(-1, 1, (m, k))
    B2 = rng.uniform(-1, 1, (k, n)) + 1j * rng.uniform(-1, 1, (k, n))
    C2 = rng.uniform(-1, 1, (m, n)) + 1j * rng.uniform(-1, 1, (m, n))
    alpha, beta = (1 + 0.5j), (0.25 - 0.75j)
    A, B = store(A2, m, np.nan), store(B2, k, np.nan)
    Cd, C4 = store(C2, m, SENTINEL), store(C2, m, SENTINEL)
    hi, S = oracle.ref_gemm_hi("N", "N", m, n, k, alpha, A, m, B, k, beta, Cd, m)
    oracle.ref_gemm("N", "N", m, n, k, alpha, A, m, B, k, beta, Cd, m)
    oracle.ref_zgemm_4m("N", "N", m, n, k, alpha, A, m, B, k, beta, C4, m)
    bound = 2 * (2 * k + 4) * 2.0 ** -53 * unstore(S, m, n, m)
    for X in (Cd, C4):
        d = unstore(X, m, n, m) - unstore(hi, m, n, m)
        assert np.all(np.abs(d.real) <= bound) and np.all(np.abs(d.imag) <= bound)
    ref_np = alpha * (A2 @ B2) + beta * C2
    assert np.allclose(unstore(hi, m, n, m), ref_np, rtol=0, atol=1e-12)


def test_complex_quick_returns(oracle):
    rng = np.random.default_rng(10)
    m, n, k = 4, 3, 5
    C2 = rng.uniform(-1, 1, (m, n)) + 1j * rng.uniform(-1, 1, (m, n))
    nanA, nanB = np.full((m, k), np.nan + 0j), np.full((k, n), np.nan + 0j)
    C = store(C2, m, SENTINEL)
    oracle.ref_gemm("N", "N", m, n, k, 0j, store(nanA, m, np.nan), m, store(nanB, k, np.nan), k, 0.5 + 0.5j, C, m)
    assert np.array_equal(unstore(C, m, n, m), (0.5 + 0.5j) * C2)
    C = store(np.full((m, n), np.nan + 0j), m, SENTINEL)
    A2 = rng.uniform(-1, 1, (m, k)) + 0j
    B2 = rng.uniform(-1, 1, (k, n)) + 0j
    oracle.ref_gemm("N", "N", m, n, k, 1 + 0j, store(A2, m, np.nan), m, store(B2, k, np.nan), k, 0j, C, m)
    assert np.all(np.isfinite(unstore(C, m, n, m)))
    with pytest.raises(ValueError):
        oracle.ref_gemm("X", "N", m, n, k, 1 + 0j, store(A2, m, np.nan), m, store(B2, k, np.nan), k, 0j, C, m)


def _zint(rng, shape):
    return (rng.integers(-4, 5, shape) + 1j * rng.integers(-4, 5, shape)).astype(np.complex128)


def _zop(X, t):
    return X if t == "N" else (X.T if t == "T" else X.conj().T)


def test_conjugate_transposes_of_the_complex_oracle(oracle):
    """'C' pinned four ways: numpy's X.conj().T on exact integer data (all nine op pairs, direct, 4M and 3M);
    'C' on X equals 'T' on conj(X) bit for bit (negation is exact); the Hermitian identity
    (A^H B)^H = B^H A bit for bit (same products, multiplication commutes, the imaginary parts are exact
    negatives); and the diagonal of A^H A has imaginary part exactly zero and a non-negative real part."""
    rng = np.random.default_rng(21)
    m, n, k = 6, 5, 7
    for ta in "NTC":
        for tb in "NTC":
            ra, ca = (m, k) if ta == "N" else (k, m)
            rb, cb = (k, n) if tb == "N" else (n, k)
            A2, B2, C2 = _zint(rng, (ra, ca)), _zint(rng, (rb, cb)), _zint(rng, (m, n))
            alpha, beta = 2 - 1j, 0.5 + 0.5j
            want = alpha * (_zop(A2, ta) @ _zop(B2, tb)) + beta * C2
            A, B = store(A2, ra + 1, np.nan), store(B2, rb + 3, np.nan)
            for fn in (oracle.ref_gemm, oracle.ref_zgemm_4m, oracle.ref_zgemm_3m):
                C = store(C2, m + 2, SENTINEL)
                fn(ta, tb, m, n, k, alpha, A, ra + 1, B, rb + 3, beta, C, m + 2)
                assert np.array_equal(unstore(C, m, n, m + 2), want), (ta, tb, fn.__name__)
                assert np.all(padding(C, m, n, m + 2).real == SENTINEL)
    # general data: C on X == T on conj(X), bitwise
    A2 = rng.uniform(-1, 1, (k, m)) + 1j * rng.uniform(-1, 1, (k, m))
    B2 = rng.uniform(-1, 1, (k, n)) + 1j * rng.uniform(-1, 1, (k, n))
    C2 = rng.uniform(-1, 1, (m, n)) + 1j * rng.uniform(-1, 1, (m, n))
    X, Y = store(C2, m, SENTINEL), store(C2, m, SENTINEL)
    oracle.ref_gemm("C", "N", m, n, k, 0.7 - 0.2j, store(A2, k, np.nan), k, store(B2, k, np.nan), k, 0.3j, X, m)
    oracle.ref_gemm("T", "N", m, n, k, 0.7 - 0.2j, store(A2.conj(), k, np.nan), k, store(B2, k, np.nan), k, 0.3j, Y, m)
    assert bits_equal(X, Y)
    # Hermitian identity, bitwise
    X, Y = store(np.zeros((m, n), complex), m, SENTINEL), store(np.zeros((n, m), complex), n, SENTINEL)
    oracle.ref_gemm("C", "N", m, n, k, 1 + 0j, store(A2, k, np.nan), k, store(B2, k, np.nan), k, 0j, X, m)
    oracle.ref_gemm("C", "N", n, m, k, 1 + 0j, store(B2, k, np.nan), k, store(A2, k, np.nan), k, 0j, Y, n)
    assert bits_equal(unstore(X, m, n, m), unstore(Y, n, m, n).conj().T)
    # Gram matrix
    G = store(np.zeros((m, m), complex), m, SENTINEL)
    oracle.ref_gemm("C", "N", m, m, k, 1 + 0j, store(A2, k, np.nan), k, store(A2, k, np.nan), k, 0j, G, m)
    d = np.diag(unstore(G, m, m, m))
    assert np.all(d.imag == 0.0) and np.all(d.real > 0.0)
    assert np.allclose(d.real, np.sum(np.abs(A2) ** 2, axis=0), rtol=1e-14)


def test_complex_wide_oracle_magnitude_sum_and_result_exact(oracle):
    """The wide complex oracle's two outputs against independent evaluations, for all nine op pairs (N/T/C).

    S, the magnitude sum every complex tolerance is built from, against exact rational arithmetic:
    S_ij = (|ar|+|ai|) sum_p (|Ar|+|Ai|)_ip (|Br|+|Bi|)_pj + (|br|+|bi|)(|Cr|+|Ci|)_ij, to 1e-12 relative; a scaled
    sum, a dropped absolute value or a forgotten alpha/beta factor all move it by far more.  Chi, the rounded wide
    result, against numpy on integer data (where the exact result is representable) bit for bit, and against the
    rational result on general data within one rounding of S."""
    rng = np.random.default_rng(31)
    m, n, k = 4, 3, 9
    F = lambda x: Fraction(float(x))
    for ta in "NTC":
        for tb in "NTC":
            ra, ca = (m, k) if ta == "N" else (k, m)
            rb, cb = (k, n) if tb == "N" else (n, k)
            A2 = rng.uniform(-1, 1, (ra, ca)) + 1j * rng.uniform(-1, 1, (ra, ca))
            B2 = rng.uniform(-1, 1, (rb, cb)) + 1j * rng.uniform(-1, 1, (rb, cb))
            C2 = rng.uniform(-1, 1, (m, n)) + 1j * rng.uniform(-1, 1, (m, n))
            alpha, beta = (0.75 - 0.5j), (-0.25 + 1.5j)
            A, B, C = store(A2, ra + 2, np.nan), store(B2, rb + 1, np.nan), store(C2, m + 3, SENTINEL)
            hi, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A, ra + 2, B, rb + 1, beta, C, m + 3)
            hi2, S2 = unstore(hi, m, n, m), unstore(S, m, n, m)
            opA, opB = _zop(A2, ta), _zop(B2, tb)
            for i in range(m):
                for j in range(n):
                    mag = sum((abs(F(opA[i, p].real)) + abs(F(opA[i, p].imag))) *
                              (abs(F(opB[p, j].real)) + abs(F(opB[p, j].imag))) for p in range(k))
                    s_exact = (abs(F(alpha.real)) + abs(F(alpha.imag))) * mag + \
                        (abs(F(beta.real)) + abs(F(beta.imag))) * (abs(F(C2[i, j].real)) + abs(F(C2[i, j].imag)))
                    assert abs(F(S2[i, j]) - s_exact) <= Fraction(1, 10 ** 12) * s_exact, (ta, tb, i, j)
                    sr = sum(F(opA[i, p].real) * F(opB[p, j].real) - F(opA[i, p].imag) * F(opB[p, j].imag)
                             for p in range(k))
                    si = sum(F(opA[i, p].real) * F(opB[p, j].imag) + F(opA[i, p].imag) * F(opB[p, j].real)
                             for p in range(k))
                    wr = F(alpha.real) * sr - F(alpha.imag) * si + F(beta.real) * F(C2[i, j].real) - \
                        F(beta.imag) * F(C2[i, j].imag)
                    wi = F(alpha.real) * si + F(alpha.imag) * sr + F(beta.real) * F(C2[i, j].imag) + \
                        F(beta.imag) * F(C2[i, j].real)
                    tol = Fraction(2.0 ** -52) * s_exact  # long double accumulation, then one rounding to double
                    assert abs(F(hi2[i, j].real) - wr) <= tol and abs(F(hi2[i, j].imag) - wi) <= tol, (ta, tb, i, j)
            # integer data: the exact result is a double, so Chi must equal numpy's bit for bit
            A2, B2, C2 = _zint(rng, (ra, ca)), _zint(rng, (rb, cb)), _zint(rng, (m, n))
            alpha, beta = 2 - 1j, 0.5 + 0.5j
            hi, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, store(A2, ra, np.nan), ra, store(B2, rb, np.nan), rb,
                                       beta, store(C2, m, SENTINEL), m)
            assert np.array_equal(unstore(hi, m, n, m), alpha * (_zop(A2, ta) @ _zop(B2, tb)) + beta * C2)
            want_s = 3.0 * ((np.abs(_zop(A2, ta).real) + np.abs(_zop(A2, ta).imag)) @
                            (np.abs(_zop(B2, tb).real) + np.abs(_zop(B2, tb).imag))) + \
                1.0 * (np.abs(C2.real) + np.abs(C2.imag))
            assert np.array_equal(unstore(S, m, n, m), want_s)  # small integers and halves: exact


def test_3m_steps_against_the_definition(oracle):
    """3M against direct complex arithmetic on general data: both components within 2*(3k+6)*u*S of the wide
    result (S = sum (|Ar|+|Ai|)(|Br|+|Bi|) scaled by |alpha| plus the beta term), and the real component, which
    3M computes exactly as 4M does, bitwise equal to 4M's."""
    rng = np.random.default_rng(22)
    m, n, k = 24, 20, 65
    for ta in "NC":
        for tb in "NT":
            ra, ca = (m, k) if ta == "N" else (k, m)
            rb, cb = (k, n) if tb == "N" else (n, k)
            A2 = rng.uniform(-1, 1, (ra, ca)) + 1j * rng.uniform(-1, 1, (ra, ca))
            B2 = rng.uniform(-1, 1, (rb, cb)) + 1j * rng.uniform(-1, 1, (rb, cb))
            C2 = rng.uniform(-1, 1, (m, n)) + 1j * rng.uniform(-1, 1, (m, n))
            alpha, beta = (1 + 0.5j), (0.25 - 0.75j)
            A, B = store(A2, ra, np.nan), store(B2, rb, np.nan)
            C3, C4, C0 = store(C2, m, SENTINEL), store(C2, m, SENTINEL), store(C2, m, SENTINEL)
            hi, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A, ra, B, rb, beta, C0, m)
            oracle.ref_zgemm_3m(ta, tb, m, n, k, alpha, A, ra, B, rb, beta, C3, m)
            oracle.ref_zgemm_4m(ta, tb, m, n, k, alpha, A, ra, B, rb, beta, C4, m)
            bound = 2 * (3 * k + 6) * 2.0 ** -53 * unstore(S, m, n, m)
            d = unstore(C3, m, n, m) - unstore(hi, m, n, m)
            assert np.all(np.abs(d.real) <= bound) and np.all(np.abs(d.imag) <= bound)
            assert bits_equal(unstore(C3, m, n, m).real.copy(), unstore(C4, m, n, m).real.copy())
            assert not bits_equal(unstore(C3, m, n, m).imag.copy(), unstore(C4, m, n, m).imag.copy())


def test_padding_of_operands_is_never_used(oracle):
    """NaN padding rows in A and B leave the result finite; changing the padding changes nothing."""
    rng = np.random.default_rng(12)
    m, n, k = 8, 6, 10
    for ta, tb in TRANS:
        (ra, ca), (rb, cb) = op_shapes(ta, tb, m, n, k)
        A2, B2 = rng.uniform(-1, 1, (ra, ca)), rng.uniform(-1, 1, (rb, cb))
        C1, C2 = np.zeros(m * n), np.zeros(m * n)
        oracle.ref_gemm(ta, tb, m, n, k, 1.0, store(A2, ra + 5, np.nan), ra + 5, store(B2, rb + 4, np.nan), rb + 4, 0.0, C1, m)
        oracle.ref_gemm(ta, tb, m, n, k, 1.0, store(A2, ra, 0.0), ra, store(B2, rb, 0.0), rb, 0.0, C2, m)
        assert np.all(np.isfinite(C1)) and bits_equal(C1, C2)


def test_argument_errors(oracle):
    z = np.zeros(64)
    bad = [
        (("X", "N", 2, 2, 2, 1.0, z, 2, z, 2, 0.0, z, 2), 1),
        (("N", "Q", 2, 2, 2, 1.0, z, 2, z, 2, 0.0, z, 2), 2),
        (("N", "N", -1, 2, 2, 1.0, z, 2, z, 2, 0.0, z, 2), 3),
        (("N", "N", 2, -1, 2, 1.0, z, 2, z, 2, 0.0, z, 2), 4),
        (("N", "N", 2, 2, -1, 1.0, z, 2, z, 2, 0.0, z, 2), 5),
        (("N", "N", 3, 2, 2, 1.0, z, 2, z, 2, 0.0, z, 3), 8),
        (("T", "N", 3, 2, 4, 1.0, z, 3, z, 4, 0.0, z, 3), 8),
        (("N", "N", 2, 2, 3, 1.0, z, 2, z, 2, 0.0, z, 2), 10),
        (("N", "T", 2, 3, 2, 1.0, z, 2, z, 2, 0.0, z, 2), 10),
        (("N", "N", 3, 2, 2, 1.0, z, 3, z, 2, 0.0, z, 2), 13),
    ]
    for args, idx in bad:
        with pytest.raises(ValueError, match=f"argument {idx}$"):
            oracle.ref_gemm(*args)
