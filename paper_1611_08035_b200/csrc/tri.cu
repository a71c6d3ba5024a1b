// Triangular level-3 routines on the GEMM kernel: TRMM (B := alpha*op(A)*B or alpha*B*op(A)) and TRSM (solve
// op(A)*X = alpha*B or X*op(A) = alpha*B), A triangular.  The paper names the level-3 BLAS as consumers of its
// GEMM kernel (Abstract, Introduction); this is the usual recursive formulation that puts almost all of the
// arithmetic into large GEMM calls:
//
//     T = [T11  0 ; T21 T22] (lower):   X1 = solve(T11, B1);  B2 := alpha*B2 - T21*X1 (GEMM);  X2 = solve(T22, B2)
//
// and its mirror images for upper triangles, the right side and the products.  The recursion stops at diagonal
// blocks of order <= 32, which a small kernel handles with one warp per right-hand side (or per row of B for
// the right side): the block of T sits in shared memory, lane i of the warp owns unknown i.
#include <cuda_runtime.h>

#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

constexpr int NB = 32;             // order of a leaf block = one warp: lane i owns unknown i
constexpr int LEAF_THREADS = 256;  // 8 warps
constexpr int LEAF_VECS = 32;      // vectors per CTA (4 per warp)

bool t_is_n(char c) { return c == 'N' || c == 'n'; }
bool t_is_t(char c) { return c == 'T' || c == 't' || c == 'C' || c == 'c'; }

// One leaf: nvec independent vectors x of length nb (element i of vector v at X[i*si + v*sv]; one of si, sv is 1)
// and the nb x nb triangular matrix M with M(i,p) = mt ? A(p,i) : A(i,p), lower triangular iff LOWER (the
// caller passes the triangle as it looks after `mt`), unit diagonal iff unit.
//   SOLVE:  x := M^-1 * (alpha*x)          else:  x := alpha * M * x
// A warp works on one vector at a time, lane i holding x_i; values travel between lanes by shuffle.  M is
// padded to 32 x 32 with the identity and x with zeros.  The CTA's 32 vectors pass through a shared-memory
// tile so that global loads and stores are coalesced whichever of si, sv is 1.
template <typename T, bool SOLVE, bool LOWER>
__global__ void __launch_bounds__(LEAF_THREADS)
    tri_leaf_kernel(int nb, const T* __restrict__ A, int64_t lda, bool mt, bool unit, T alpha, T* __restrict__ X,
                    int64_t si, int64_t sv, int64_t nvec) {
  __shared__ T Ms[NB * NB];               // Ms[p*NB + i] = M(i, p): a column of M is contiguous over lanes
  __shared__ T Xs[LEAF_VECS * (NB + 1)];  // Xs[v*(NB+1) + i]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < NB * NB; e += LEAF_THREADS) {
    const int i = e / NB, p = e % NB;  // logical M(i, p)
    T v = (i == p) ? T(1) : T(0);
    if (i < nb && p < nb) {
      if (i == p) {
        if (!unit) v = A[i + (int64_t)i * lda];
      } else if (LOWER ? (i > p) : (i < p)) {
        v = mt ? A[p + (int64_t)i * lda] : A[i + (int64_t)p * lda];
      }
    }
    Ms[p * NB + i] = v;
  }
  const int64_t v0 = blockIdx.x * (int64_t)LEAF_VECS;
  const bool elem_fastest = (si == 1);  // consecutive threads walk along whichever index is contiguous in memory
  for (int e = tid; e < LEAF_VECS * NB; e += LEAF_THREADS) {
    const int v = elem_fastest ? e / NB : e % LEAF_VECS, i = elem_fastest ? e % NB : e / LEAF_VECS;
    T val = T(0);
    if (i < nb && v0 + v < nvec) val = X[i * si + (v0 + v) * sv];
    Xs[v * (NB + 1) + i] = val;
  }
  __syncthreads();

  const T diag = Ms[lane * NB + lane];
  for (int v = warp; v < LEAF_VECS; v += LEAF_THREADS / 32) {
    T x = Xs[v * (NB + 1) + lane];
    if (SOLVE) {
      x = alpha * x;
#pragma unroll 4
      for (int s = 0; s < NB; ++s) {
        const int i = LOWER ? s : NB - 1 - s;  // forward for a lower M, backward for an upper one
        if (lane == i) x = x / diag;
        const T xi = __shfl_sync(0xffffffffu, x, i);
        if (LOWER ? (lane > i) : (lane < i)) x -= Ms[i * NB + lane] * xi;  // M(lane, i)
      }
    } else {
      T acc = T(0);
#pragma unroll 4
      for (int p = 0; p < NB; ++p) {
        const T xp = __shfl_sync(0xffffffffu, x, p);
        if (LOWER ? (p <= lane) : (p >= lane)) acc += Ms[p * NB + lane] * xp;  // M(lane, p)
      }
      x = alpha * acc;
    }
    Xs[v * (NB + 1) + lane] = x;
  }
  __syncthreads();
  for (int e = tid; e < LEAF_VECS * NB; e += LEAF_THREADS) {
    const int v = elem_fastest ? e / NB : e % LEAF_VECS, i = elem_fastest ? e % NB : e / LEAF_VECS;
    if (i < nb && v0 + v < nvec) X[i * si + (v0 + v) * sv] = Xs[v * (NB + 1) + i];
  }
}

template <typename T>
struct Tri {
  bool right, lower, tr, unit, solve;
  const T* A;
  int64_t lda;
  T* B;
  int64_t ldb;
  int64_t m, n;
  cudaStream_t st;
  int rc = B2_OK;

  bool eff_lower() const { return lower != tr; }  // op(A) is lower triangular

  // block T[r0:r0+rows, c0:c0+cols] of T = op(A) as a GEMM operand: pointer and transpose character
  const T* t_block(int64_t r0, int64_t c0, char* op) const {
    *op = tr ? 'T' : 'N';
    return tr ? A + c0 + r0 * lda : A + r0 + c0 * lda;
  }

  void leaf(int64_t o, int64_t nb, T alpha) {
    if (rc) return;
    const T* Ab = A + o + o * lda;
    // left: vectors are columns of B, M = op(A) block.  right: vectors are rows, M = (op(A) block)^T.
    const bool mt = right ? !tr : tr;
    const bool m_lower = right ? !eff_lower() : eff_lower();
    T* X = right ? B + o * ldb : B + o;
    const int64_t si = right ? ldb : 1, sv = right ? 1 : ldb, nvec = right ? m : n;
    const unsigned grid = (unsigned)((nvec + LEAF_VECS - 1) / LEAF_VECS);
    if (solve) {
      if (m_lower)
        tri_leaf_kernel<T, true, true><<<grid, LEAF_THREADS, 0, st>>>((int)nb, Ab, lda, mt, unit, alpha, X, si, sv, nvec);
      else
        tri_leaf_kernel<T, true, false><<<grid, LEAF_THREADS, 0, st>>>((int)nb, Ab, lda, mt, unit, alpha, X, si, sv, nvec);
    } else {
      if (m_lower)
        tri_leaf_kernel<T, false, true><<<grid, LEAF_THREADS, 0, st>>>((int)nb, Ab, lda, mt, unit, alpha, X, si, sv, nvec);
      else
        tri_leaf_kernel<T, false, false><<<grid, LEAF_THREADS, 0, st>>>((int)nb, Ab, lda, mt, unit, alpha, X, si, sv, nvec);
    }
    if (cudaGetLastError() != cudaSuccess) rc = B2_ERR_LAUNCH;
  }

  // Block update with the off-diagonal block of T: dst := ga * (T-block product with src) + gb * dst, where for
  // the left side dst/src are row blocks of B and for the right side column blocks.
  //   left:  dst = B[d0:d0+dn, :],  src = B[s0:s0+sn, :],  dst += T[d0.., s0..] * src
  //   right: dst = B[:, d0:d0+dn],  src = B[:, s0:s0+sn],  dst += src * T[s0.., d0..]
  void update(int64_t d0, int64_t dn, int64_t s0, int64_t sn, T ga, T gb) {
    if (rc) return;
    char op;
    if (!right) {
      const T* Tb = t_block(d0, s0, &op);
      rc = gemm_entry<T>(B2_VARIANT_AUTO, op, 'N', dn, n, sn, ga, Tb, lda, B + s0, ldb, gb, B + d0, ldb, st);
    } else {
      const T* Tb = t_block(s0, d0, &op);
      rc = gemm_entry<T>(B2_VARIANT_AUTO, 'N', op, m, dn, sn, ga, B + s0 * ldb, ldb, Tb, lda, gb, B + d0 * ldb, ldb, st);
    }
  }

  // order [o, o+na) of the triangular matrix
  void run(int64_t o, int64_t na, T alpha) {
    if (rc || na <= 0) return;
    if (na <= NB) {
      leaf(o, na, alpha);
      return;
    }
    const int64_t h = ((na / 2 + NB - 1) / NB) * NB;  // first part: a multiple of the leaf order
    const int64_t o2 = o + h, n2 = na - h;
    // Which half is independent of the other?  In T*X (left) row block 1 involves only T11 when T is lower;
    // in X*T (right) column block 1 involves only T11 when T is upper.
    const bool first_is_free = right ? !eff_lower() : eff_lower();
    if (solve) {
      if (first_is_free) {  // X1 first, then block 2 := alpha*B2 - (T21*X1 or X1*T12)
        run(o, h, alpha);
        update(o2, n2, o, h, T(-1), alpha);
        run(o2, n2, T(1));
      } else {
        run(o2, n2, alpha);
        update(o, h, o2, n2, T(-1), alpha);
        run(o, h, T(1));
      }
    } else {
      if (first_is_free) {  // block 2 of the product needs the old block 1: finish block 2 first
        run(o2, n2, alpha);
        update(o2, n2, o, h, alpha, T(1));
        run(o, h, alpha);
      } else {
        run(o, h, alpha);
        update(o, h, o2, n2, alpha, T(1));
        run(o2, n2, alpha);
      }
    }
  }
};

template <typename T>
int tri_entry(bool solve, char side, char uplo, char trans, char diag, int64_t m, int64_t n, T alpha, const T* A,
              int64_t lda, T* B, int64_t ldb, void* cuda_stream) {
  const bool left = (side == 'L' || side == 'l'), right = (side == 'R' || side == 'r');
  const bool lower = (uplo == 'L' || uplo == 'l'), upper = (uplo == 'U' || uplo == 'u');
  const bool unit = (diag == 'U' || diag == 'u'), nonunit = (diag == 'N' || diag == 'n');
  if (!left && !right) return -1;
  if (!lower && !upper) return -2;
  if (!t_is_n(trans) && !t_is_t(trans)) return -3;
  if (!unit && !nonunit) return -4;
  if (m < 0) return -5;
  if (n < 0) return -6;
  const int64_t na = left ? m : n;
  const bool nonempty = m > 0 && n > 0;
  if (nonempty && alpha != T(0) && !A) return -8;
  if (lda < (na > 1 ? na : 1)) return -9;
  if (nonempty && !B) return -10;
  if (ldb < (m > 1 ? m : 1)) return -11;
  if (!nonempty) return B2_OK;
  if (alpha == T(0))  // B := 0, A is not referenced
    return gemm_entry<T>(B2_VARIANT_AUTO, 'N', 'N', m, n, 0, T(0), nullptr, m, nullptr, 1, T(0), B, ldb, cuda_stream);
  Tri<T> t;
  t.right = right, t.lower = lower, t.tr = t_is_t(trans), t.unit = unit, t.solve = solve;
  t.A = A, t.lda = lda, t.B = B, t.ldb = ldb, t.m = m, t.n = n, t.st = (cudaStream_t)cuda_stream;
  t.run(0, na, alpha);
  return t.rc;
}

}  // namespace
}  // namespace b2

extern "C" int b2_dtrsm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, double alpha,
                        const double* A, int64_t lda, double* B, int64_t ldb, void* cuda_stream) {
  return b2::tri_entry<double>(true, side, uplo, transa, diag, m, n, alpha, A, lda, B, ldb, cuda_stream);
}
extern "C" int b2_strsm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, float alpha,
                        const float* A, int64_t lda, float* B, int64_t ldb, void* cuda_stream) {
  return b2::tri_entry<float>(true, side, uplo, transa, diag, m, n, alpha, A, lda, B, ldb, cuda_stream);
}
extern "C" int b2_dtrmm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, double alpha,
                        const double* A, int64_t lda, double* B, int64_t ldb, void* cuda_stream) {
  return b2::tri_entry<double>(false, side, uplo, transa, diag, m, n, alpha, A, lda, B, ldb, cuda_stream);
}
extern "C" int b2_strmm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, float alpha,
                        const float* A, int64_t lda, float* B, int64_t ldb, void* cuda_stream) {
  return b2::tri_entry<float>(false, side, uplo, transa, diag, m, n, alpha, A, lda, B, ldb, cuda_stream);
}
