/*
 * CPU oracle for GEMM -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may call this file.
 * It shares no code with the CUDA library and neither includes the other.
 *
 * What it computes.  The paper's micro-kernel (Section 2.1, "The micro-kernel") is the sum
 * of rank-1 updates  C += sum_{p<k} a_p b_p^T.  The method reaches, up to the order of the
 * floating-point summation, the plain definition of that sum, so the oracle is the
 * definition written out, with the scaling, transposition and leading dimensions of the
 * level-3 BLAS statement (which the paper does not restate):
 *
 *     acc_ij = sum_{p=0}^{k-1} op(A)_ip * op(B)_pj        (ascending p)
 *     C_ij   = alpha * acc_ij + beta * C_ij
 *     op(X) = X or X^T,   column-major  X(r,c) = X[r + c*ldx].
 *
 * Rules kept here so a reader can check it by eye:
 *   - one multiply and one add per term, in the working precision, p ascending, starting
 *     from zero (compile with -ffp-contract=off: no fused multiply-add, no fast-math);
 *   - beta == 0: C is not read (C_ij = alpha*acc_ij);  alpha == 0 or k == 0: A and B are not
 *     read (C_ij = beta*C_ij, or 0 when beta == 0);  alpha == 0 and beta == 1: nothing;
 *   - only entries (i<m, j<n) of C are touched; padding rows of A, B, C are never read;
 *   - the only parallelism is OpenMP over columns j, which changes no element's arithmetic;
 *   - `cols`/`ncols` restrict the work to a list of columns j (NULL = all n columns).
 *
 * The *_hi variants accumulate in a wider type (long double for fp64 data, double for fp32
 * data), return the result in that wider type's nearest working-precision value, and also
 * return the magnitude sum used by forward error bounds,
 *     S_ij = |alpha| * sum_p |op(A)_ip| |op(B)_pj| + |beta| |C_ij|.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static int is_trans(char t) { return t == 'T' || t == 't' || t == 'C' || t == 'c'; }
static int is_notrans(char t) { return t == 'N' || t == 'n'; }
static int is_conj(char t) { return t == 'C' || t == 'c'; } /* complex data only; for real data 'C' is 'T' */

/* BLAS argument check; returns 0 or the 1-based index of the first illegal argument. */
static int check_args(char ta, char tb, int64_t m, int64_t n, int64_t k, int64_t lda, int64_t ldb, int64_t ldc) {
  if (!is_trans(ta) && !is_notrans(ta)) return 1;
  if (!is_trans(tb) && !is_notrans(tb)) return 2;
  if (m < 0) return 3;
  if (n < 0) return 4;
  if (k < 0) return 5;
  int64_t rows_a = is_notrans(ta) ? m : k, rows_b = is_notrans(tb) ? k : n;
  if (lda < (rows_a > 1 ? rows_a : 1)) return 8;
  if (ldb < (rows_b > 1 ? rows_b : 1)) return 10;
  if (ldc < (m > 1 ? m : 1)) return 13;
  return 0;
}

#define DEFINE_REF_GEMM(NAME, T)                                                                          \
  int NAME(char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A, int64_t lda,    \
           const T* B, int64_t ldb, T beta, T* C, int64_t ldc, const int64_t* cols, int64_t ncols) {       \
    int bad = check_args(transa, transb, m, n, k, lda, ldb, ldc);                                          \
    if (bad) return -bad;                                                                                  \
    if (m == 0 || n == 0) return 0;                                                                        \
    if ((alpha == (T)0 || k == 0) && beta == (T)1) return 0;                                               \
    const int ta = is_trans(transa), tb = is_trans(transb);                                                \
    const int scale_only = (alpha == (T)0 || k == 0);                                                      \
    const int64_t nj = cols ? ncols : n;                                                                   \
    _Pragma("omp parallel for schedule(dynamic, 1)") for (int64_t jj = 0; jj < nj; ++jj) {                 \
      const int64_t j = cols ? cols[jj] : jj;                                                              \
      for (int64_t i = 0; i < m; ++i) {                                                                    \
        T acc = (T)0;                                                                                      \
        if (!scale_only) {                                                                                 \
          for (int64_t p = 0; p < k; ++p) {                                                                \
            const T a = ta ? A[p + i * lda] : A[i + p * lda];                                              \
            const T b = tb ? B[j + p * ldb] : B[p + j * ldb];                                              \
            const T prod = a * b;                                                                          \
            acc = acc + prod;                                                                              \
          }                                                                                                \
        }                                                                                                  \
        T* c = &C[i + j * ldc];                                                                            \
        if (scale_only) {                                                                                  \
          *c = (beta == (T)0) ? (T)0 : beta * *c;                                                          \
        } else if (beta == (T)0) {                                                                         \
          *c = alpha * acc;                                                                                \
        } else {                                                                                           \
          const T t1 = alpha * acc;                                                                        \
          const T t2 = beta * *c;                                                                          \
          *c = t1 + t2;                                                                                    \
        }                                                                                                  \
      }                                                                                                    \
    }                                                                                                      \
    return 0;                                                                                              \
  }

DEFINE_REF_GEMM(ref_dgemm, double)
DEFINE_REF_GEMM(ref_sgemm, float)

/* Wide-accumulation variants; Chi receives the rounded wide result, S the magnitude sum. */
#define DEFINE_REF_GEMM_HI(NAME, T, W, ABSW)                                                              \
  int NAME(char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A, int64_t lda,    \
           const T* B, int64_t ldb, T beta, const T* C, int64_t ldc, T* Chi, double* S, int64_t ldo,       \
           const int64_t* cols, int64_t ncols) {                                                           \
    int bad = check_args(transa, transb, m, n, k, lda, ldb, ldc);                                          \
    if (bad) return -bad;                                                                                  \
    if (ldo < (m > 1 ? m : 1)) return -15;                                                                 \
    if (m == 0 || n == 0) return 0;                                                                        \
    const int ta = is_trans(transa), tb = is_trans(transb);                                                \
    const int64_t nj = cols ? ncols : n;                                                                   \
    _Pragma("omp parallel for schedule(dynamic, 1)") for (int64_t jj = 0; jj < nj; ++jj) {                 \
      const int64_t j = cols ? cols[jj] : jj;                                                              \
      for (int64_t i = 0; i < m; ++i) {                                                                    \
        W acc = 0, mag = 0;                                                                                \
        if (alpha != (T)0) {                                                                               \
          for (int64_t p = 0; p < k; ++p) {                                                                \
            const W a = ta ? A[p + i * lda] : A[i + p * lda];                                              \
            const W b = tb ? B[j + p * ldb] : B[p + j * ldb];                                              \
            acc += a * b;                                                                                  \
            mag += ABSW(a) * ABSW(b);                                                                      \
          }                                                                                                \
        }                                                                                                  \
        W r = (W)alpha * acc, s = ABSW((W)alpha) * mag;                                                    \
        if (beta != (T)0) {                                                                                \
          r += (W)beta * (W)C[i + j * ldc];                                                                \
          s += ABSW((W)beta) * ABSW((W)C[i + j * ldc]);                                                    \
        }                                                                                                  \
        Chi[i + j * ldo] = (T)r;                                                                           \
        S[i + j * ldo] = (double)s;                                                                        \
      }                                                                                                    \
    }                                                                                                      \
    return 0;                                                                                              \
  }

DEFINE_REF_GEMM_HI(ref_dgemm_hi, double, long double, fabsl)
DEFINE_REF_GEMM_HI(ref_sgemm_hi, float, double, fabs)

/*
 * Complex double GEMM by direct complex arithmetic (interleaved re,im; ld in complex
 * elements).  Each term is the textbook product (ar*br - ai*bi, ar*bi + ai*br) added to the
 * running sum; the epilogue is the complex alpha*acc + beta*C.  transa/transb: N, T (plain
 * transpose) or C (conjugate transpose: the transposed element with its imaginary part
 * negated).
 * The paper names complex GEMM only as a consumer of the real kernel (Abstract).
 */
int ref_zgemm(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A,
              int64_t lda, const double* B, int64_t ldb, const double* beta, double* C, int64_t ldc,
              const int64_t* cols, int64_t ncols) {
  int bad = check_args(transa, transb, m, n, k, lda, ldb, ldc);
  if (bad) return -bad;
  if (m == 0 || n == 0) return 0;
  /* op(X) = X^H for 'C': the element is read transposed and its imaginary part negated (exact) */
  const double ca = is_conj(transa) ? -1.0 : 1.0, cb = is_conj(transb) ? -1.0 : 1.0;
  const double alr = alpha[0], ali = alpha[1], ber = beta[0], bei = beta[1];
  const int alpha0 = (alr == 0.0 && ali == 0.0), beta0 = (ber == 0.0 && bei == 0.0);
  if ((alpha0 || k == 0) && ber == 1.0 && bei == 0.0) return 0;
  const int ta = is_trans(transa), tb = is_trans(transb);
  const int64_t nj = cols ? ncols : n;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t jj = 0; jj < nj; ++jj) {
    const int64_t j = cols ? cols[jj] : jj;
    for (int64_t i = 0; i < m; ++i) {
      double sr = 0.0, si = 0.0;
      if (!alpha0) {
        for (int64_t p = 0; p < k; ++p) {
          const double* a = ta ? &A[2 * (p + i * lda)] : &A[2 * (i + p * lda)];
          const double* b = tb ? &B[2 * (j + p * ldb)] : &B[2 * (p + j * ldb)];
          const double are = a[0], aim = ca * a[1], bre = b[0], bim = cb * b[1];
          const double pr = are * bre - aim * bim;
          const double pi = are * bim + aim * bre;
          sr = sr + pr;
          si = si + pi;
        }
      }
      double* c = &C[2 * (i + j * ldc)];
      double rr = 0.0, ri = 0.0;
      if (!alpha0) {
        rr = alr * sr - ali * si;
        ri = alr * si + ali * sr;
      }
      if (!beta0) {
        const double cr = c[0], ci = c[1];
        rr = rr + (ber * cr - bei * ci);
        ri = ri + (ber * ci + bei * cr);
      }
      c[0] = rr;
      c[1] = ri;
    }
  }
  return 0;
}

/* Wide (long double) complex GEMM; Chi = rounded result, S = one magnitude sum per element:
 *   S_ij = (|alr|+|ali|) * sum_p (|Ar|+|Ai|)_ip (|Br|+|Bi|)_pj + (|ber|+|bei|) (|Cr|+|Ci|)_ij,
 * an upper bound on the magnitude sums of both the real and the imaginary component. */
int ref_zgemm_hi(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A,
                 int64_t lda, const double* B, int64_t ldb, const double* beta, const double* C, int64_t ldc,
                 double* Chi, double* S, int64_t ldo, const int64_t* cols, int64_t ncols) {
  int bad = check_args(transa, transb, m, n, k, lda, ldb, ldc);
  if (bad) return -bad;
  if (ldo < (m > 1 ? m : 1)) return -16;
  const double ca = is_conj(transa) ? -1.0 : 1.0, cb = is_conj(transb) ? -1.0 : 1.0;
  if (m == 0 || n == 0) return 0;
  const long double alr = alpha[0], ali = alpha[1], ber = beta[0], bei = beta[1];
  const int alpha0 = (alr == 0 && ali == 0), beta0 = (ber == 0 && bei == 0);
  const int ta = is_trans(transa), tb = is_trans(transb);
  const int64_t nj = cols ? ncols : n;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t jj = 0; jj < nj; ++jj) {
    const int64_t j = cols ? cols[jj] : jj;
    for (int64_t i = 0; i < m; ++i) {
      long double sr = 0, si = 0, mag = 0;
      if (!alpha0) {
        for (int64_t p = 0; p < k; ++p) {
          const double* a = ta ? &A[2 * (p + i * lda)] : &A[2 * (i + p * lda)];
          const double* b = tb ? &B[2 * (j + p * ldb)] : &B[2 * (p + j * ldb)];
          const long double ar = a[0], ai = ca * a[1], br = b[0], bi = cb * b[1];
          sr += ar * br - ai * bi;
          si += ar * bi + ai * br;
          mag += (fabsl(ar) + fabsl(ai)) * (fabsl(br) + fabsl(bi));
        }
      }
      long double rr = alr * sr - ali * si, ri = alr * si + ali * sr;
      long double s = (fabsl(alr) + fabsl(ali)) * mag;
      if (!beta0) {
        const long double cr = C[2 * (i + j * ldc)], ci = C[2 * (i + j * ldc) + 1];
        rr += ber * cr - bei * ci;
        ri += ber * ci + bei * cr;
        s += (fabsl(ber) + fabsl(bei)) * (fabsl(cr) + fabsl(ci));
      }
      Chi[2 * (i + j * ldo)] = (double)rr;
      Chi[2 * (i + j * ldo) + 1] = (double)ri;
      S[i + j * ldo] = (double)s;
    }
  }
  return 0;
}

/* Number of OpenMP threads a parallel region would use (reported beside CPU timings). */
#ifdef _OPENMP
#include <omp.h>
int ref_num_threads(void) { return omp_get_max_threads(); }
#else
int ref_num_threads(void) { return 1; }
#endif

/*
 * TF32 tensor-core variants of the fp32 GEMM (reported separately from the FP32-FMA entry; the paper has no
 * counterpart, the definitions follow the published TF32 format: 1 sign, 8 exponent, 10 mantissa bits).
 *
 *   ref_tf32_round   x rounded to the nearest TF32 value, ties away from zero (the conversion the packing
 *                    kernel applies, PTX cvt.rna.tf32.f32).
 *   ref_sgemm_tf32   terms == 1:  acc_ij = sum_p t(a_ip) t(b_pj)                       ("TF32 x1")
 *                    terms == 3:  a = ah + al with ah = t(a), al = t(a - ah) (likewise b),
 *                                 acc_ij = sum_p (ah bh + ah bl + al bh)               ("3 x TF32")
 *                    evaluated in double (every product of two TF32 values is exact in double), then
 *                    Cout_ij = fp32(alpha*acc_ij + beta*C_ij), and S_ij = |alpha| sum_p |a_ip||b_pj| + |beta||C_ij|.
 */
float ref_tf32_round(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return x; /* Inf, NaN unchanged */
  u += 0x00001000u;                               /* half of the last kept place, magnitude-wise */
  u &= 0xffffe000u;
  memcpy(&x, &u, 4);
  return x;
}

int ref_sgemm_tf32(int terms, char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                   int64_t lda, const float* B, int64_t ldb, float beta, const float* C, int64_t ldc, float* Cout,
                   double* S, int64_t ldo, const int64_t* cols, int64_t ncols) {
  if (terms != 1 && terms != 3) return -1;
  int bad = check_args(transa, transb, m, n, k, lda, ldb, ldc);
  if (bad) return -bad - 1;
  if (ldo < (m > 1 ? m : 1)) return -17;
  if (m == 0 || n == 0) return 0;
  const int ta = is_trans(transa), tb = is_trans(transb);
  const int64_t nj = cols ? ncols : n;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t jj = 0; jj < nj; ++jj) {
    const int64_t j = cols ? cols[jj] : jj;
    for (int64_t i = 0; i < m; ++i) {
      double acc = 0.0, mag = 0.0;
      if (alpha != 0.0f) {
        for (int64_t p = 0; p < k; ++p) {
          const float a = ta ? A[p + i * lda] : A[i + p * lda];
          const float b = tb ? B[j + p * ldb] : B[p + j * ldb];
          const float ah = ref_tf32_round(a), bh = ref_tf32_round(b);
          if (terms == 1) {
            acc += (double)ah * (double)bh;
          } else {
            const float al = ref_tf32_round(a - ah), bl = ref_tf32_round(b - bh);
            acc += (double)ah * (double)bh + (double)ah * (double)bl + (double)al * (double)bh;
          }
          mag += fabs((double)a) * fabs((double)b);
        }
      }
      double r = (double)alpha * acc, s = fabs((double)alpha) * mag;
      if (beta != 0.0f) {
        r += (double)beta * (double)C[i + j * ldc];
        s += fabs((double)beta) * fabs((double)C[i + j * ldc]);
      }
      Cout[i + j * ldo] = (float)r;
      S[i + j * ldo] = s;
    }
  }
  return 0;
}

/*
 * Symmetric rank-k update, the level-3 routine that is a GEMM restricted to one triangle (the paper names the
 * level-3 BLAS as consumers of the GEMM kernel, Abstract and Introduction; the definition is the BLAS one):
 *     trans = N:  C := alpha * A * A^T + beta * C,   A is n x k
 *     trans = T:  C := alpha * A^T * A + beta * C,   A is k x n
 * Only the triangle named by uplo ('L': i >= j, 'U': i <= j) of the n x n matrix C is read or written.
 * Same arithmetic rules as ref_*gemm: ascending p, one multiply and one add per term, beta == 0 does not read C,
 * alpha == 0 or k == 0 scales the triangle only.
 */
#define DEFINE_REF_SYRK(NAME, T)                                                                          \
  int NAME(char uplo, char trans, int64_t n, int64_t k, T alpha, const T* A, int64_t lda, T beta, T* C,   \
           int64_t ldc) {                                                                                  \
    const int lower = (uplo == 'L' || uplo == 'l'), upper = (uplo == 'U' || uplo == 'u');                  \
    if (!lower && !upper) return -1;                                                                       \
    if (!is_trans(trans) && !is_notrans(trans)) return -2;                                                 \
    if (n < 0) return -3;                                                                                  \
    if (k < 0) return -4;                                                                                  \
    const int tr = is_trans(trans);                                                                        \
    const int64_t rows_a = tr ? k : n;                                                                     \
    if (lda < (rows_a > 1 ? rows_a : 1)) return -7;                                                        \
    if (ldc < (n > 1 ? n : 1)) return -10;                                                                 \
    if (n == 0) return 0;                                                                                  \
    const int scale_only = (alpha == (T)0 || k == 0);                                                      \
    if (scale_only && beta == (T)1) return 0;                                                              \
    _Pragma("omp parallel for schedule(dynamic, 1)") for (int64_t j = 0; j < n; ++j) {                     \
      const int64_t i_lo = lower ? j : 0, i_hi = lower ? n : j + 1;                                        \
      for (int64_t i = i_lo; i < i_hi; ++i) {                                                              \
        T acc = (T)0;                                                                                      \
        if (!scale_only) {                                                                                 \
          for (int64_t p = 0; p < k; ++p) {                                                                \
            const T a = tr ? A[p + i * lda] : A[i + p * lda];                                              \
            const T b = tr ? A[p + j * lda] : A[j + p * lda];                                              \
            const T prod = a * b;                                                                          \
            acc = acc + prod;                                                                              \
          }                                                                                                \
        }                                                                                                  \
        T* c = &C[i + j * ldc];                                                                            \
        if (scale_only) {                                                                                  \
          *c = (beta == (T)0) ? (T)0 : beta * *c;                                                          \
        } else if (beta == (T)0) {                                                                         \
          *c = alpha * acc;                                                                                \
        } else {                                                                                           \
          const T t1 = alpha * acc;                                                                        \
          const T t2 = beta * *c;                                                                          \
          *c = t1 + t2;                                                                                    \
        }                                                                                                  \
      }                                                                                                    \
    }                                                                                                      \
    return 0;                                                                                              \
  }

DEFINE_REF_SYRK(ref_dsyrk, double)
DEFINE_REF_SYRK(ref_ssyrk, float)

/*
 * Triangular level-3 routines (the paper names the level-3 BLAS as consumers of the GEMM kernel, Abstract and
 * Introduction; their definitions are the BLAS ones).  A is a triangular matrix of order na (= m for side 'L',
 * n for side 'R'); only the triangle named by uplo is read, and with diag = 'U' its diagonal is taken as 1
 * without being read.  T = op(A) below is that triangular matrix, transposed for trans = 'T'.
 *
 *   TRMM:  B := alpha * T * B   (side L)      or   B := alpha * B * T   (side R)
 *          every element is the sum over the non-zero part of the row/column of T, ascending index, one multiply
 *          and one add per term, then one multiply by alpha.  Evaluated from a copy of B (the routine is in place).
 *
 *   TRSM:  solve T * X = alpha * B (side L)   or   X * T = alpha * B (side R);  X overwrites B.
 *          Substitution, one unknown after the other in the order the triangle dictates:
 *              x_i = (alpha * b_i - sum_{p already solved} T_ip x_p) / T_ii      (side L; side R alike on rows)
 *          the sum taken in ascending p with one multiply and one add per term, subtracted once from alpha*b_i,
 *          then one division (none for diag = 'U').  alpha == 0 gives X = 0 without reading A.
 *
 * t_elem returns T(i, p) for an effective position, 0 outside the triangle, 1 on a unit diagonal.
 */
#define DEFINE_REF_TRI(SUFFIX, T)                                                                          \
  static T t_elem_##SUFFIX(const T* A, int64_t lda, int lower, int tr, int unit, int64_t i, int64_t p) {    \
    /* (i, p) indexes T = op(A); the stored element is A(i, p) or, transposed, A(p, i) */                   \
    const int64_t r = tr ? p : i, c = tr ? i : p;                                                           \
    if (r == c) return unit ? (T)1 : A[r + c * lda];                                                        \
    if (lower ? (r > c) : (r < c)) return A[r + c * lda];                                                   \
    return (T)0;                                                                                            \
  }                                                                                                         \
  static int check_tri_##SUFFIX(char side, char uplo, char trans, char diag, int64_t m, int64_t n,          \
                                int64_t lda, int64_t ldb) {                                                 \
    const int left = (side == 'L' || side == 'l'), right = (side == 'R' || side == 'r');                    \
    if (!left && !right) return 1;                                                                          \
    if (!(uplo == 'L' || uplo == 'l' || uplo == 'U' || uplo == 'u')) return 2;                              \
    if (!is_trans(trans) && !is_notrans(trans)) return 3;                                                   \
    if (!(diag == 'U' || diag == 'u' || diag == 'N' || diag == 'n')) return 4;                              \
    if (m < 0) return 5;                                                                                    \
    if (n < 0) return 6;                                                                                    \
    const int64_t na = left ? m : n;                                                                        \
    if (lda < (na > 1 ? na : 1)) return 9;                                                                  \
    if (ldb < (m > 1 ? m : 1)) return 11;                                                                   \
    return 0;                                                                                               \
  }                                                                                                         \
  int ref_##SUFFIX##trmm(char side, char uplo, char trans, char diag, int64_t m, int64_t n, T alpha,        \
                         const T* A, int64_t lda, T* B, int64_t ldb) {                                      \
    const int bad = check_tri_##SUFFIX(side, uplo, trans, diag, m, n, lda, ldb);                            \
    if (bad) return -bad;                                                                                   \
    if (m == 0 || n == 0) return 0;                                                                         \
    const int left = (side == 'L' || side == 'l'), lower = (uplo == 'L' || uplo == 'l');                    \
    const int tr = is_trans(trans), unit = (diag == 'U' || diag == 'u');                                    \
    if (alpha == (T)0) {                                                                                    \
      for (int64_t j = 0; j < n; ++j)                                                                       \
        for (int64_t i = 0; i < m; ++i) B[i + j * ldb] = (T)0;                                              \
      return 0;                                                                                             \
    }                                                                                                       \
    T* old = (T*)malloc(sizeof(T) * (size_t)m * (size_t)n);                                                 \
    if (!old) return -100;                                                                                  \
    for (int64_t j = 0; j < n; ++j)                                                                         \
      for (int64_t i = 0; i < m; ++i) old[i + j * m] = B[i + j * ldb];                                      \
    const int eff_lower = (lower != tr); /* op(A) is lower triangular */                                    \
    _Pragma("omp parallel for schedule(dynamic, 1)") for (int64_t j = 0; j < n; ++j) {                      \
      for (int64_t i = 0; i < m; ++i) {                                                                     \
        T acc = (T)0;                                                                                       \
        if (left) { /* sum_p T(i,p) old(p,j): p <= i for lower T, p >= i for upper */                       \
          const int64_t lo = eff_lower ? 0 : i, hi = eff_lower ? i + 1 : m;                                 \
          for (int64_t p = lo; p < hi; ++p) {                                                               \
            const T prod = t_elem_##SUFFIX(A, lda, lower, tr, unit, i, p) * old[p + j * m];                 \
            acc = acc + prod;                                                                               \
          }                                                                                                 \
        } else { /* sum_p old(i,p) T(p,j): p >= j for lower T, p <= j for upper */                          \
          const int64_t lo = eff_lower ? j : 0, hi = eff_lower ? n : j + 1;                                 \
          for (int64_t p = lo; p < hi; ++p) {                                                               \
            const T prod = old[i + p * m] * t_elem_##SUFFIX(A, lda, lower, tr, unit, p, j);                 \
            acc = acc + prod;                                                                               \
          }                                                                                                 \
        }                                                                                                   \
        B[i + j * ldb] = alpha * acc;                                                                       \
      }                                                                                                     \
    }                                                                                                       \
    free(old);                                                                                              \
    return 0;                                                                                               \
  }                                                                                                         \
  int ref_##SUFFIX##trsm(char side, char uplo, char trans, char diag, int64_t m, int64_t n, T alpha,        \
                         const T* A, int64_t lda, T* B, int64_t ldb) {                                      \
    const int bad = check_tri_##SUFFIX(side, uplo, trans, diag, m, n, lda, ldb);                            \
    if (bad) return -bad;                                                                                   \
    if (m == 0 || n == 0) return 0;                                                                         \
    const int left = (side == 'L' || side == 'l'), lower = (uplo == 'L' || uplo == 'l');                    \
    const int tr = is_trans(trans), unit = (diag == 'U' || diag == 'u');                                    \
    if (alpha == (T)0) {                                                                                    \
      for (int64_t j = 0; j < n; ++j)                                                                       \
        for (int64_t i = 0; i < m; ++i) B[i + j * ldb] = (T)0;                                              \
      return 0;                                                                                             \
    }                                                                                                       \
    const int eff_lower = (lower != tr);                                                                    \
    if (left) { /* columns of B are independent systems T x = alpha b */                                    \
      _Pragma("omp parallel for schedule(dynamic, 1)") for (int64_t j = 0; j < n; ++j) {                    \
        T* x = &B[j * ldb];                                                                                 \
        for (int64_t s = 0; s < m; ++s) {                                                                   \
          const int64_t i = eff_lower ? s : m - 1 - s; /* forward for lower T, backward for upper */        \
          const int64_t lo = eff_lower ? 0 : i + 1, hi = eff_lower ? i : m;                                 \
          T acc = (T)0;                                                                                     \
          for (int64_t p = lo; p < hi; ++p) {                                                               \
            const T prod = t_elem_##SUFFIX(A, lda, lower, tr, unit, i, p) * x[p];                           \
            acc = acc + prod;                                                                               \
          }                                                                                                 \
          const T rhs = alpha * x[i];                                                                       \
          T v = rhs - acc;                                                                                  \
          if (!unit) v = v / t_elem_##SUFFIX(A, lda, lower, tr, unit, i, i);                                \
          x[i] = v;                                                                                         \
        }                                                                                                   \
      }                                                                                                     \
    } else { /* rows of B are independent systems x^T T = alpha b^T: x_j needs x_p with T(p,j) != 0 */      \
      _Pragma("omp parallel for schedule(dynamic, 16)") for (int64_t i = 0; i < m; ++i) {                   \
        for (int64_t s = 0; s < n; ++s) {                                                                   \
          const int64_t j = eff_lower ? n - 1 - s : s; /* upper T: forward over columns; lower: backward */ \
          const int64_t lo = eff_lower ? j + 1 : 0, hi = eff_lower ? n : j;                                 \
          T acc = (T)0;                                                                                     \
          for (int64_t p = lo; p < hi; ++p) {                                                               \
            const T prod = B[i + p * ldb] * t_elem_##SUFFIX(A, lda, lower, tr, unit, p, j);                 \
            acc = acc + prod;                                                                               \
          }                                                                                                 \
          const T rhs = alpha * B[i + j * ldb];                                                             \
          T v = rhs - acc;                                                                                  \
          if (!unit) v = v / t_elem_##SUFFIX(A, lda, lower, tr, unit, j, j);                                \
          B[i + j * ldb] = v;                                                                               \
        }                                                                                                   \
      }                                                                                                     \
    }                                                                                                       \
    return 0;                                                                                               \
  }

DEFINE_REF_TRI(d, double)
DEFINE_REF_TRI(s, float)
