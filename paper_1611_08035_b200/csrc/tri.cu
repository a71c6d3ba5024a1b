// Triangular level-3 routines on the GEMM kernel: TRMM (B := alpha*op(A)*B or alpha*B*op(A)) and TRSM (solve
// op(A)*X = alpha*B or X*op(A) = alpha*B), A triangular.  The paper names the level-3 BLAS as consumers of its
// GEMM kernel (Abstract, Introduction); this is the usual recursive formulation that puts almost all of the
// arithmetic into large GEMM calls:
//
//     T = [T11  0 ; T21 T22] (lower):   X1 = solve(T11, B1);  B2 := alpha*B2 - T21*X1 (GEMM);  X2 = solve(T22, B2)
//
// and its mirror images for upper triangles, the right side and the products.  The recursion stops at diagonal
// blocks of order <= 128, which a small kernel handles with one warp per four right-hand sides (or rows of B
// for the right side), 32 x 32 sub-block by sub-block.
#include <cuda_runtime.h>

#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

constexpr int SUB = 32;            // a sub-block = one warp: lane i owns unknown i of the sub-block
constexpr int NSUB = 4;            // sub-blocks per leaf
constexpr int NB = SUB * NSUB;     // order of a leaf block (128)
constexpr int LEAF_THREADS = 256;  // 8 warps
constexpr int VPW = 4;             // vectors per warp
constexpr int LEAF_VECS = VPW * LEAF_THREADS / 32;  // vectors per CTA (32)

bool t_is_n(char c) { return c == 'N' || c == 'n'; }
bool t_is_t(char c) { return c == 'T' || c == 't' || c == 'C' || c == 'c'; }

// One leaf: nvec independent vectors x of length nb <= 128 (element i of vector v at X[i*si + v*sv]; one of si,
// sv is 1) and the nb x nb triangular matrix M with M(i,p) = mt ? A(p,i) : A(i,p), lower triangular iff LOWER
// (the caller passes the triangle as it looks after `mt`), unit diagonal iff unit.
//   SOLVE:  x := M^-1 * (alpha*x)          else:  x := alpha * M * x
// M is handled as 4 x 4 sub-blocks of order 32.  A warp holds four vectors, lane i owning element i of each
// sub-block (16 values per lane); values travel between lanes by shuffle.  The CTA walks through the sub-blocks
// of the triangle in dependency order -- solve (or multiply by) a diagonal sub-block, then apply the
// off-diagonal sub-blocks of its block column (row) -- staging one 32 x 32 sub-block of M at a time in shared
// memory.  M is padded with the identity and x with zeros beyond nb; sub-blocks wholly beyond nb are skipped.
// The CTA's 32 vectors pass through a shared-memory tile so that global loads and stores are coalesced
// whichever of si, sv is 1.
template <typename T, bool SOLVE, bool LOWER>
__global__ void __launch_bounds__(LEAF_THREADS, 2)
    tri_leaf_kernel(int nb, const T* __restrict__ A, int64_t lda, bool mt, bool unit, T alpha, T* __restrict__ X,
                    int64_t si, int64_t sv, int64_t nvec) {
  __shared__ T Ms[SUB * SUB];             // Ms[p*SUB + i] = M(i, p) of the staged sub-block
  __shared__ T Xs[LEAF_VECS * (NB + 1)];  // Xs[v*(NB+1) + i]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nsub = (nb + SUB - 1) / SUB;  // sub-blocks that hold anything

  // Sub-block (bi, bj) of M travels global -> registers (fetch, issued one step ahead so that its latency hides
  // behind the arithmetic of the current step) -> shared memory (commit, between two barriers).
  constexpr int PER_THREAD = SUB * SUB / LEAF_THREADS;
  T staged[PER_THREAD];
  auto fetch = [&](int bi, int bj) {
#pragma unroll
    for (int u = 0; u < PER_THREAD; ++u) {
      const int e = tid + u * LEAF_THREADS;
      const int i = e % SUB, p = e / SUB;
      const int gi = bi * SUB + i, gp = bj * SUB + p;
      T v = (gi == gp) ? T(1) : T(0);
      if (gi < nb && gp < nb) {
        if (gi == gp) {
          if (!unit) v = A[gi + (int64_t)gi * lda];
        } else if (LOWER ? (gi > gp) : (gi < gp)) {
          v = mt ? A[gp + (int64_t)gi * lda] : A[gi + (int64_t)gp * lda];
        }
      }
      staged[u] = v;
    }
  };
  auto commit = [&]() {
    __syncthreads();  // everybody is done with the previous sub-block
#pragma unroll
    for (int u = 0; u < PER_THREAD; ++u) Ms[tid + u * LEAF_THREADS] = staged[u];  // index p*SUB + i
    __syncthreads();
  };

  const int64_t v0 = blockIdx.x * (int64_t)LEAF_VECS;
  const bool elem_fastest = (si == 1);  // consecutive threads walk along whichever index is contiguous in memory
  for (int e = tid; e < LEAF_VECS * NB; e += LEAF_THREADS) {
    const int v = elem_fastest ? e / NB : e % LEAF_VECS, i = elem_fastest ? e % NB : e / LEAF_VECS;
    T val = T(0);
    if (i < nb && v0 + v < nvec) val = X[i * si + (v0 + v) * sv];
    Xs[v * (NB + 1) + i] = val;
  }
  __syncthreads();

  T x[VPW][NSUB];
#pragma unroll
  for (int q = 0; q < VPW; ++q)
#pragma unroll
    for (int b = 0; b < NSUB; ++b) x[q][b] = Xs[(warp * VPW + q) * (NB + 1) + b * SUB + lane];
  if (SOLVE) {
#pragma unroll
    for (int q = 0; q < VPW; ++q)
#pragma unroll
      for (int b = 0; b < NSUB; ++b) x[q][b] = alpha * x[q][b];
  }

  // Steps (sb, tb), tb >= sb.  SOLVE: sub-block blk(sb) is solved at tb == sb, then leaves sub-block blk(tb).
  // Product: row blk(sb) is formed from its diagonal sub-block (tb == sb) and the sub-blocks blk(tb) whose old
  // values it still needs; a lower M goes bottom-up so that those are still unchanged.
  auto blk = [](int s) { return (SOLVE == LOWER) ? s : NSUB - 1 - s; };
  auto fetch_step = [&](int sb, int tb) {
    if (SOLVE) fetch(blk(tb), blk(sb)); else fetch(blk(sb), blk(tb));
  };
  T acc[VPW];
  fetch_step(0, 0);
#pragma unroll
  for (int sb = 0; sb < NSUB; ++sb) {
#pragma unroll
    for (int tb = sb; tb < NSUB; ++tb) {
      commit();
      if (tb + 1 < NSUB) fetch_step(sb, tb + 1);
      else if (sb + 1 < NSUB) fetch_step(sb + 1, sb + 1);
      const int bs = blk(sb), bt = blk(tb);
      if (bs >= nsub || bt >= nsub) continue;  // nothing but padding (uniform over the CTA)
      if (SOLVE) {
        if (tb == sb) {
          const T diag = Ms[lane * SUB + lane];
#pragma unroll 2
          for (int s = 0; s < SUB; ++s) {
            const int i = LOWER ? s : SUB - 1 - s;  // forward within a lower sub-block, backward within an upper
            const T mi = Ms[i * SUB + lane];        // M(lane, i)
#pragma unroll
            for (int q = 0; q < VPW; ++q) {         // four independent chains
              if (lane == i) x[q][bs] = x[q][bs] / diag;
              const T xi = __shfl_sync(0xffffffffu, x[q][bs], i);
              if (LOWER ? (lane > i) : (lane < i)) x[q][bs] -= mi * xi;
            }
          }
        } else {
#pragma unroll
          for (int q = 0; q < VPW; ++q) acc[q] = T(0);
#pragma unroll 4
          for (int p = 0; p < SUB; ++p) {
            const T mp = Ms[p * SUB + lane];  // M(lane of sub-block bt, p of sub-block bs)
#pragma unroll
            for (int q = 0; q < VPW; ++q) acc[q] += mp * __shfl_sync(0xffffffffu, x[q][bs], p);
          }
#pragma unroll
          for (int q = 0; q < VPW; ++q) x[q][bt] -= acc[q];
        }
      } else {
        if (tb == sb) {
#pragma unroll
          for (int q = 0; q < VPW; ++q) acc[q] = T(0);
        }
#pragma unroll 4
        for (int p = 0; p < SUB; ++p) {
          const T mp = Ms[p * SUB + lane];
          const bool inside = (tb != sb) || (LOWER ? (p <= lane) : (p >= lane));
#pragma unroll
          for (int q = 0; q < VPW; ++q) {
            const T xp = __shfl_sync(0xffffffffu, x[q][bt], p);
            if (inside) acc[q] += mp * xp;
          }
        }
      }
    }
    if (!SOLVE && blk(sb) < nsub) {
#pragma unroll
      for (int q = 0; q < VPW; ++q) x[q][blk(sb)] = alpha * acc[q];
    }
  }

#pragma unroll
  for (int q = 0; q < VPW; ++q)
#pragma unroll
    for (int b = 0; b < NSUB; ++b) Xs[(warp * VPW + q) * (NB + 1) + b * SUB + lane] = x[q][b];
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
