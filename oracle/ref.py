"""numpy front end of the C oracle (``ref_gemm.c``) -- TEST INFRASTRUCTURE, not the product.

Matrices are passed the way BLAS sees them: a flat numpy array holding column-major storage
plus a leading dimension, X(r, c) = X[r + c*ldx].  Real arrays are float64 or float32; complex
arrays are complex128 (interleaved re, im; leading dimensions in complex elements).

  ref_gemm      the definition in working precision (Section 2.1 sum of rank-1 updates with the
                BLAS alpha/beta/op/ld semantics); updates C in place.
  ref_gemm_hi   the same sum accumulated in a wider type, plus the magnitude sum S used by
                forward error bounds; returns (C_hi, S) and leaves C untouched.
  ref_zgemm_4m  complex GEMM assembled from four calls of the real oracle on split planes (the
                4M formulation), used to check that formulation against direct complex arithmetic.
"""
from __future__ import annotations

import ctypes
from ctypes import c_char, c_double, c_float, c_int, c_int64, c_void_p

import numpy as np

from . import build as _build

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(_build.build()))
        real_tail = [c_char, c_char, c_int64, c_int64, c_int64]
        _lib.ref_dgemm.argtypes = real_tail + [c_double, c_void_p, c_int64, c_void_p, c_int64, c_double, c_void_p,
                                               c_int64, c_void_p, c_int64]
        _lib.ref_sgemm.argtypes = real_tail + [c_float, c_void_p, c_int64, c_void_p, c_int64, c_float, c_void_p,
                                               c_int64, c_void_p, c_int64]
        _lib.ref_dgemm_hi.argtypes = real_tail + [c_double, c_void_p, c_int64, c_void_p, c_int64, c_double, c_void_p,
                                                  c_int64, c_void_p, c_void_p, c_int64, c_void_p, c_int64]
        _lib.ref_sgemm_hi.argtypes = real_tail + [c_float, c_void_p, c_int64, c_void_p, c_int64, c_float, c_void_p,
                                                  c_int64, c_void_p, c_void_p, c_int64, c_void_p, c_int64]
        _lib.ref_zgemm.argtypes = real_tail + [c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_void_p,
                                               c_int64, c_void_p, c_int64]
        _lib.ref_zgemm_hi.argtypes = real_tail + [c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_void_p,
                                                  c_int64, c_void_p, c_void_p, c_int64, c_void_p, c_int64]
        _lib.ref_tf32_round.argtypes = [c_float]
        _lib.ref_tf32_round.restype = c_float
        _lib.ref_sgemm_tf32.argtypes = [c_int] + real_tail + [c_float, c_void_p, c_int64, c_void_p, c_int64, c_float,
                                                              c_void_p, c_int64, c_void_p, c_void_p, c_int64, c_void_p,
                                                              c_int64]
        _lib.ref_sgemm_tf32.restype = c_int
        _lib.ref_dsyrk.argtypes = [c_char, c_char, c_int64, c_int64, c_double, c_void_p, c_int64, c_double, c_void_p, c_int64]
        _lib.ref_ssyrk.argtypes = [c_char, c_char, c_int64, c_int64, c_float, c_void_p, c_int64, c_float, c_void_p, c_int64]
        _lib.ref_dsyrk.restype = _lib.ref_ssyrk.restype = c_int
        tri = [c_char, c_char, c_char, c_char, c_int64, c_int64]
        _lib.ref_dtrmm.argtypes = _lib.ref_dtrsm.argtypes = tri + [c_double, c_void_p, c_int64, c_void_p, c_int64]
        _lib.ref_strmm.argtypes = _lib.ref_strsm.argtypes = tri + [c_float, c_void_p, c_int64, c_void_p, c_int64]
        for fn in ("ref_dtrmm", "ref_dtrsm", "ref_strmm", "ref_strsm"):
            getattr(_lib, fn).restype = c_int
        for fn in ("ref_dgemm", "ref_sgemm", "ref_dgemm_hi", "ref_sgemm_hi", "ref_zgemm", "ref_zgemm_hi",
                   "ref_num_threads"):
            getattr(_lib, fn).restype = c_int
    return _lib


def num_threads() -> int:
    """OpenMP threads the oracle uses."""
    return lib().ref_num_threads()


def _tr(c: str) -> bytes:
    return c.encode("ascii")[:1]


def _flat(x: np.ndarray, dtype) -> np.ndarray:
    if not isinstance(x, np.ndarray) or x.dtype != dtype or x.ndim != 1 or not x.flags.c_contiguous:
        raise TypeError(f"expected a flat contiguous numpy array of {dtype}")
    return x


def _need(x: np.ndarray, ld: int, ncols: int, nrows: int, what: str) -> None:
    if ncols > 0 and nrows > 0 and x.size < ld * (ncols - 1) + nrows:
        raise ValueError(f"{what}: storage of {x.size} elements is too small for ld={ld}, {nrows}x{ncols}")


def _cols(cols):
    if cols is None:
        return None, 0, None
    arr = np.ascontiguousarray(np.asarray(cols, dtype=np.int64))
    return arr.ctypes.data, arr.size, arr


def _check_storage(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, read_ab):
    ta, tb = transa in "TtCc", transb in "TtCc"
    if read_ab:
        _need(A, lda, m if ta else k, k if ta else m, "A")
        _need(B, ldb, k if tb else n, n if tb else k, "B")
    _need(C, ldc, n, m, "C")


def ref_gemm(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cols=None) -> None:
    """C := alpha*op(A)*op(B) + beta*C by the plain definition; C (flat storage) is updated in place."""
    dt = C.dtype
    if dt == np.complex128:
        al = np.array([complex(alpha).real, complex(alpha).imag], dtype=np.float64)
        be = np.array([complex(beta).real, complex(beta).imag], dtype=np.float64)
        fn, args_a, args_b = lib().ref_zgemm, al.ctypes.data, be.ctypes.data
        read_ab = not (al[0] == 0 and al[1] == 0) and k > 0
    elif dt == np.float64:
        fn, args_a, args_b = lib().ref_dgemm, float(alpha), float(beta)
        read_ab = alpha != 0 and k > 0
    elif dt == np.float32:
        fn, args_a, args_b = lib().ref_sgemm, float(np.float32(alpha)), float(np.float32(beta))
        read_ab = np.float32(alpha) != 0 and k > 0
    else:
        raise TypeError(f"unsupported dtype {dt}")
    _flat(A, dt), _flat(B, dt), _flat(C, dt)
    cptr, ncols, keep = _cols(cols)
    rc = fn(_tr(transa), _tr(transb), m, n, k, args_a, A.ctypes.data, lda, B.ctypes.data, ldb, args_b, C.ctypes.data,
            ldc, cptr, ncols)
    if rc != 0:
        raise ValueError(f"oracle rejected argument {-rc}")
    if m > 0 and n > 0:
        _check_storage(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, read_ab)
    del keep


def ref_gemm_hi(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cols=None):
    """Wide-accumulation result and magnitude sum S; returns (C_hi, S) as flat arrays with leading dimension m.

    For complex data C_hi is complex128 and S holds one bound term per element (valid for both components).
    Columns outside `cols` are left as NaN.
    """
    dt = C.dtype
    _flat(A, dt), _flat(B, dt), _flat(C, dt)
    ldo = max(1, m)
    Chi = np.full(ldo * max(n, 1), np.nan, dtype=dt)
    S = np.full(ldo * max(n, 1), np.nan, dtype=np.float64)
    cptr, ncols, keep = _cols(cols)
    if m > 0 and n > 0:
        _check_storage(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, True)
    if dt == np.complex128:
        al = np.array([complex(alpha).real, complex(alpha).imag], dtype=np.float64)
        be = np.array([complex(beta).real, complex(beta).imag], dtype=np.float64)
        rc = lib().ref_zgemm_hi(_tr(transa), _tr(transb), m, n, k, al.ctypes.data, A.ctypes.data, lda, B.ctypes.data,
                                ldb, be.ctypes.data, C.ctypes.data, ldc, Chi.ctypes.data, S.ctypes.data, ldo, cptr,
                                ncols)
    elif dt == np.float64:
        rc = lib().ref_dgemm_hi(_tr(transa), _tr(transb), m, n, k, float(alpha), A.ctypes.data, lda, B.ctypes.data,
                                ldb, float(beta), C.ctypes.data, ldc, Chi.ctypes.data, S.ctypes.data, ldo, cptr, ncols)
    elif dt == np.float32:
        rc = lib().ref_sgemm_hi(_tr(transa), _tr(transb), m, n, k, float(np.float32(alpha)), A.ctypes.data, lda,
                                B.ctypes.data, ldb, float(np.float32(beta)), C.ctypes.data, ldc, Chi.ctypes.data,
                                S.ctypes.data, ldo, cptr, ncols)
    else:
        raise TypeError(f"unsupported dtype {dt}")
    if rc != 0:
        raise ValueError(f"oracle rejected argument {-rc}")
    del keep
    return Chi, S


def _split_planes(transa, transb, alpha, beta, A, B, C):
    """Real and imaginary planes for the 4M / 3M step oracles: A' = alpha*op-conjugated A, B, beta*C.

    A conjugate transpose becomes a plain transpose of the conjugated matrix (negating the imaginary plane is
    exact); returns (apr, api, br, bi, cr, ci, first_beta, ta, tb) with ta/tb the real transposes to use."""
    alpha, beta = complex(alpha), complex(beta)
    _flat(A, np.complex128), _flat(B, np.complex128), _flat(C, np.complex128)
    Av = A.view(np.float64)
    ar, ai = Av[0::2], Av[1::2]
    if transa in "Cc":
        ai = -ai
    apr = np.ascontiguousarray(alpha.real * ar - alpha.imag * ai)
    api = np.ascontiguousarray(alpha.real * ai + alpha.imag * ar)
    Bv = B.view(np.float64)
    br, bi = np.ascontiguousarray(Bv[0::2]), np.ascontiguousarray(Bv[1::2])
    if transb in "Cc":
        bi = -bi
    Cv = C.view(np.float64)
    cr0, ci0 = Cv[0::2].copy(), Cv[1::2].copy()
    if beta == 0:
        cr, ci, first_beta = np.zeros_like(cr0), np.zeros_like(ci0), 0.0
    else:
        cr = np.ascontiguousarray(beta.real * cr0 - beta.imag * ci0)
        ci = np.ascontiguousarray(beta.real * ci0 + beta.imag * cr0)
        first_beta = 1.0
    ta = "N" if transa in "Nn" else "T"
    tb = "N" if transb in "Nn" else "T"
    return apr, api, br, bi, cr, ci, first_beta, ta, tb


def _store_planes(C, cr, ci, m, n, ldc):
    Cv = C.view(np.float64)
    for j in range(n):  # write back only the m x n entries the operation owns
        s = slice(j * ldc, j * ldc + m)
        Cv[0::2][s] = cr[s]
        Cv[1::2][s] = ci[s]


def ref_zgemm_4m(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc) -> None:
    """Complex GEMM from four real-oracle calls on split planes (4M); C complex128 flat, updated in place.

    A' = alpha*A is formed elementwise in complex arithmetic (each component rounded once), then
        Cr = A'r*Br - A'i*Bi + (beta*C)r,     Ci = A'r*Bi + A'i*Br + (beta*C)i,
    each right-hand side evaluated as two real GEMM calls: (alpha=1, beta=0 or 1) followed by
    (alpha=-1 or +1, beta=1).  With beta == 0 the old C is not read.  Conjugate transposes negate the
    imaginary plane of that operand first.
    """
    apr, api, br, bi, cr, ci, first_beta, ta, tb = _split_planes(transa, transb, alpha, beta, A, B, C)
    ref_gemm(ta, tb, m, n, k, 1.0, apr, lda, br, ldb, first_beta, cr, ldc)
    ref_gemm(ta, tb, m, n, k, -1.0, api, lda, bi, ldb, 1.0, cr, ldc)
    ref_gemm(ta, tb, m, n, k, 1.0, apr, lda, bi, ldb, first_beta, ci, ldc)
    ref_gemm(ta, tb, m, n, k, 1.0, api, lda, br, ldb, 1.0, ci, ldc)
    _store_planes(C, cr, ci, m, n, ldc)


def ref_zgemm_3m(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc) -> None:
    """Complex GEMM from three real products (3M), the steps in this order; C complex128 flat, updated in place.

        A' = alpha*A (as in 4M);  As = A'r + A'i,  Bs = Br + Bi     (one rounding per element)
        T1 = A'r*Br,  T2 = A'i*Bi                                    (real GEMMs, beta = 0)
        Cr = ((beta*C)r + T1) - T2
        Ci = (((beta*C)i - T1) - T2) + As*Bs                         (last step: real GEMM with beta = 1)

    The imaginary part is the difference of larger numbers, so its error is bounded relative to
    sum (|Ar|+|Ai|)(|Br|+|Bi|), not to the magnitude of the imaginary products alone.
    """
    apr, api, br, bi, cr, ci, first_beta, ta, tb = _split_planes(transa, transb, alpha, beta, A, B, C)
    a_sum = np.ascontiguousarray(apr + api)
    b_sum = np.ascontiguousarray(br + bi)
    t1 = np.zeros_like(cr)
    t2 = np.zeros_like(cr)
    ref_gemm(ta, tb, m, n, k, 1.0, apr, lda, br, ldb, 0.0, t1, ldc)
    ref_gemm(ta, tb, m, n, k, 1.0, api, lda, bi, ldb, 0.0, t2, ldc)
    cr = (cr + t1) - t2
    ci = np.ascontiguousarray((ci - t1) - t2)
    ref_gemm(ta, tb, m, n, k, 1.0, a_sum, lda, b_sum, ldb, 1.0, ci, ldc)
    _store_planes(C, cr, ci, m, n, ldc)


def tf32_round(x: float) -> float:
    """x (fp32) rounded to the nearest TF32 value (10 mantissa bits), ties away from zero."""
    return float(lib().ref_tf32_round(float(np.float32(x))))


def ref_sgemm_tf32(terms, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cols=None):
    """TF32 x1 (terms=1) or 3xTF32 (terms=3) GEMM by the definition, evaluated in double; returns (C_out fp32, S).

    C is not modified.  C_out and S are flat with leading dimension max(1, m); columns outside `cols` are NaN."""
    _flat(A, np.float32), _flat(B, np.float32), _flat(C, np.float32)
    ldo = max(1, m)
    out = np.full(ldo * max(n, 1), np.nan, dtype=np.float32)
    S = np.full(ldo * max(n, 1), np.nan, dtype=np.float64)
    if m > 0 and n > 0:
        _check_storage(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, True)
    cptr, ncols, keep = _cols(cols)
    rc = lib().ref_sgemm_tf32(terms, _tr(transa), _tr(transb), m, n, k, float(np.float32(alpha)), A.ctypes.data, lda,
                              B.ctypes.data, ldb, float(np.float32(beta)), C.ctypes.data, ldc, out.ctypes.data,
                              S.ctypes.data, ldo, cptr, ncols)
    if rc != 0:
        raise ValueError(f"oracle rejected argument {-rc}")
    del keep
    return out, S


def ref_syrk(uplo, trans, n, k, alpha, A, lda, beta, C, ldc) -> None:
    """C := alpha*A*A^T + beta*C (trans N) or alpha*A^T*A + beta*C (trans T) on the uplo triangle of C, in place."""
    dt = C.dtype
    _flat(A, dt), _flat(C, dt)
    if dt == np.float64:
        fn, a, b = lib().ref_dsyrk, float(alpha), float(beta)
    elif dt == np.float32:
        fn, a, b = lib().ref_ssyrk, float(np.float32(alpha)), float(np.float32(beta))
    else:
        raise TypeError(f"unsupported dtype {dt}")
    if n > 0:
        _need(C, ldc, n, n, "C")
        if alpha != 0 and k > 0:
            tr = trans in "TtCc"
            _need(A, lda, n if tr else k, k if tr else n, "A")
    rc = fn(_tr(uplo), _tr(trans), n, k, a, A.ctypes.data, lda, b, C.ctypes.data, ldc)
    if rc != 0:
        raise ValueError(f"oracle rejected argument {-rc}")


def ref_gemm_strided_batched(transa, transb, m, n, k, alpha, A, lda, stride_a, B, ldb, stride_b, beta, C, ldc,
                             stride_c, batch) -> None:
    """`batch` independent GEMMs on operands that start stride_* elements apart: one ref_gemm call per problem."""
    for b in range(batch):
        ref_gemm(transa, transb, m, n, k, alpha, A[b * stride_a:], lda, B[b * stride_b:], ldb, beta,
                 C[b * stride_c:], ldc)


def _tri_call(which, side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb) -> None:
    dt = B.dtype
    _flat(A, dt), _flat(B, dt)
    if dt == np.float64:
        fn, a = getattr(lib(), f"ref_d{which}"), float(alpha)
    elif dt == np.float32:
        fn, a = getattr(lib(), f"ref_s{which}"), float(np.float32(alpha))
    else:
        raise TypeError(f"unsupported dtype {dt}")
    if m > 0 and n > 0:
        _need(B, ldb, n, m, "B")
        if alpha != 0:
            na = m if side in "Ll" else n
            _need(A, lda, na, na, "A")
    rc = fn(_tr(side), _tr(uplo), _tr(trans), _tr(diag), m, n, a, A.ctypes.data, lda, B.ctypes.data, ldb)
    if rc != 0:
        raise ValueError(f"oracle rejected argument {-rc}")


def ref_trmm(side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb) -> None:
    """B := alpha*op(A)*B (side L) or alpha*B*op(A) (side R), A triangular; B (flat storage) updated in place."""
    _tri_call("trmm", side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb)


def ref_trsm(side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb) -> None:
    """Solve op(A)*X = alpha*B (side L) or X*op(A) = alpha*B (side R) by substitution; X overwrites B."""
    _tri_call("trsm", side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb)
