"""Pins of the TF32 oracle: the rounding against closed forms of the published format (10 mantissa bits, ties
away from zero), the x1 sum against exact rational arithmetic on rounded inputs, the 3-term split against the
fp32 oracle (it recovers fp32 accuracy up to the dropped low*low term), integer inputs exactly."""
from fractions import Fraction

import numpy as np

from helpers import SENTINEL, store, unstore


def test_tf32_round_closed_forms(oracle):
    t = oracle.tf32_round
    assert t(1.0) == 1.0 and t(-2.5) == -2.5 and t(0.0) == 0.0
    assert t(1 + 2.0 ** -10) == 1 + 2.0 ** -10          # representable
    assert t(1 + 2.0 ** -11) == 1 + 2.0 ** -10          # tie goes away from zero
    assert t(-(1 + 2.0 ** -11)) == -(1 + 2.0 ** -10)
    assert t(1 + 2.0 ** -11 - 2.0 ** -23) == 1.0         # just below the tie rounds down
    assert t(1 + 2.0 ** -11 + 2.0 ** -23) == 1 + 2.0 ** -10
    assert t(2 - 2.0 ** -23) == 2.0                      # carries into the exponent
    assert np.isinf(t(float("inf"))) and np.isnan(t(float("nan")))
    rng = np.random.default_rng(0)
    for x in rng.uniform(-4, 4, 2000).astype(np.float32):
        y = t(float(x))
        fy, fx = Fraction(y), Fraction(float(x))
        e = int(np.frexp(np.float32(abs(x)))[1]) - 1 if x != 0 else 0   # |x| in [2^e, 2^(e+1))
        ulp = Fraction(2) ** (e - 10)
        assert abs(fy - fx) <= ulp / 2                   # nearest
        assert (fy / ulp).denominator == 1               # on the TF32 grid of that binade (or the next power of two)


def test_tf32_x1_matches_rational_on_rounded_inputs(oracle):
    rng = np.random.default_rng(1)
    m, n, k = 5, 4, 19
    for ta in "NT":
        for tb in "NT":
            ra, ca = (m, k) if ta == "N" else (k, m)
            rb, cb = (k, n) if tb == "N" else (n, k)
            A2 = rng.uniform(-1, 1, (ra, ca)).astype(np.float32)
            B2 = rng.uniform(-1, 1, (rb, cb)).astype(np.float32)
            C2 = rng.uniform(-1, 1, (m, n)).astype(np.float32)
            out, S = oracle.ref_sgemm_tf32(1, ta, tb, m, n, k, 0.75, store(A2, ra + 1, np.nan), ra + 1,
                                           store(B2, rb + 2, np.nan), rb + 2, -0.5, store(C2, m + 3, SENTINEL), m + 3)
            opA = A2 if ta == "N" else A2.T
            opB = B2 if tb == "N" else B2.T
            got = unstore(out, m, n, m)
            for i in range(m):
                for j in range(n):
                    acc = sum(Fraction(oracle.tf32_round(float(opA[i, p]))) * Fraction(oracle.tf32_round(float(opB[p, j])))
                              for p in range(k))
                    exact = Fraction(0.75) * acc + Fraction(-0.5) * Fraction(float(C2[i, j]))
                    assert got[i, j] == np.float32(float(exact))  # double evaluation is exact here up to the final rounding
                    s = 0.75 * sum(abs(float(opA[i, p])) * abs(float(opB[p, j])) for p in range(k)) + 0.5 * abs(float(C2[i, j]))
                    assert abs(unstore(S, m, n, m)[i, j] - s) <= 1e-12 * s


def test_tf32_error_levels_against_fp32(oracle):
    """x1 differs from the fp32 result by about 2^-11 relative to S per operand rounding; the 3-term split is back at
    the fp32 level (the dropped low*low term is 2^-22 relative)."""
    rng = np.random.default_rng(2)
    m, n, k = 40, 30, 257
    A = store(rng.uniform(-1, 1, (m, k)).astype(np.float32), m, np.nan)
    B = store(rng.uniform(-1, 1, (k, n)).astype(np.float32), k, np.nan)
    C = store(rng.uniform(-1, 1, (m, n)).astype(np.float32), m, SENTINEL)
    hi, S = oracle.ref_gemm_hi("N", "N", m, n, k, 1.0, A, m, B, k, 0.5, C, m)
    x1, S1 = oracle.ref_sgemm_tf32(1, "N", "N", m, n, k, 1.0, A, m, B, k, 0.5, C, m)
    x3, _ = oracle.ref_sgemm_tf32(3, "N", "N", m, n, k, 1.0, A, m, B, k, 0.5, C, m)
    assert np.allclose(S, S1, rtol=1e-12)
    e1 = np.abs(x1.astype(np.float64) - hi.astype(np.float64)) / S
    e3 = np.abs(x3.astype(np.float64) - hi.astype(np.float64)) / S
    assert e1.max() <= 2.0 ** -10 and e1.max() > 2.0 ** -16       # two operand roundings of 2^-11 each
    assert e3.max() <= 2.0 ** -21                                 # fp32 level


def test_tf32_integer_inputs_exact(oracle):
    rng = np.random.default_rng(3)
    m, n, k = 17, 13, 300
    Ai, Bi, Ci = rng.integers(-4, 5, (k, m)), rng.integers(-4, 5, (k, n)), rng.integers(-4, 5, (m, n))
    for terms in (1, 3):
        out, _ = oracle.ref_sgemm_tf32(terms, "T", "N", m, n, k, 1.5, store(Ai.astype(np.float32), k, np.nan), k,
                                       store(Bi.astype(np.float32), k, np.nan), k, 0.5,
                                       store(Ci.astype(np.float32), m, SENTINEL), m)
        want = (3 * (Ai.T @ Bi) + Ci) / 2.0
        assert np.array_equal(unstore(out, m, n, m).astype(np.float64), want)
