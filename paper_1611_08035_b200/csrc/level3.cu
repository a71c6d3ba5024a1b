// Level-3 routines built on the GEMM kernel (the paper's Abstract and Introduction name the level-3 BLAS as
// its consumers): the symmetric rank-k update, which is a GEMM with op(B) = op(A)^T restricted to one triangle of
// C, the strided-batched GEMM, which is the GEMM grid replicated along grid.y, and a split-K GEMM for small
// m*n with long k, which is a batched GEMM over k-chunks followed by an ordered sum.
#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

bool l3_is_n(char c) { return c == 'N' || c == 'n'; }
bool l3_is_t(char c) { return c == 'T' || c == 't' || c == 'C' || c == 'c'; }

// C := beta*C on one triangle (tri = 1: i >= j, 2: i <= j); beta == 0 stores zeros without reading.
template <typename T>
__global__ void tri_scale_kernel(int64_t n, T beta, T* C, int64_t ldc, int tri) {
  const int64_t total = n * n;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx % n, j = idx / n;
    if (tri == 1 ? i >= j : i <= j) {
      T* c = C + i + j * ldc;
      *c = (beta == T(0)) ? T(0) : beta * *c;
    }
  }
}

// C_b := beta*C_b for every problem of a batch.
template <typename T>
__global__ void batch_scale_kernel(int64_t m, int64_t n, T beta, T* C, int64_t ldc, int64_t stride_c) {
  T* Cb = C + (int64_t)blockIdx.y * stride_c;
  const int64_t total = m * n;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx % m, j = idx / m;
    T* c = Cb + i + j * ldc;
    *c = (beta == T(0)) ? T(0) : beta * *c;
  }
}

unsigned blocks_for(int64_t total) {
  int64_t b = (total + 255) / 256;
  const int64_t cap = (int64_t)sm_count_cached() * 16;
  if (b > cap) b = cap;
  return (unsigned)(b < 1 ? 1 : b);
}

template <typename T>
int syrk(char uplo, char trans, int64_t n, int64_t k, T alpha, const T* A, int64_t lda, T beta, T* C, int64_t ldc,
         void* cuda_stream) {
  const bool lower = (uplo == 'L' || uplo == 'l'), upper = (uplo == 'U' || uplo == 'u');
  if (!lower && !upper) return -1;
  if (!l3_is_n(trans) && !l3_is_t(trans)) return -2;
  if (n < 0) return -3;
  if (k < 0) return -4;
  const bool tr = l3_is_t(trans);
  const bool scale_only = (alpha == T(0) || k == 0);
  const int64_t rows_a = tr ? k : n;
  if (n > 0 && !scale_only && !A) return -6;
  if (lda < (rows_a > 1 ? rows_a : 1)) return -7;
  if (n > 0 && !C) return -9;
  if (ldc < (n > 1 ? n : 1)) return -10;
  if (n == 0) return B2_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int tri = lower ? 1 : 2;
  if (scale_only) {
    if (beta == T(1)) return B2_OK;
    tri_scale_kernel<T><<<blocks_for(n * n), 256, 0, st>>>(n, beta, C, ldc, tri);
    return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }
  GemmExtra ex;
  ex.tri = tri;
  // op(A) * op(A)^T: the second operand is the same array with the opposite transpose
  return gemm_launch_checked<T>(B2_VARIANT_AUTO, tr, !tr, n, n, k, alpha, A, lda, A, lda, beta, C, ldc, ex, st);
}

template <typename T>
int gemm_strided_batched(char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A, int64_t lda,
                         int64_t stride_a, const T* B, int64_t ldb, int64_t stride_b, T beta, T* C, int64_t ldc,
                         int64_t stride_c, int64_t batch, void* cuda_stream) {
  if (!l3_is_n(transa) && !l3_is_t(transa)) return -1;
  if (!l3_is_n(transb) && !l3_is_t(transb)) return -2;
  if (m < 0) return -3;
  if (n < 0) return -4;
  if (k < 0) return -5;
  const bool scale_only = (alpha == T(0) || k == 0);
  const bool nonempty = m > 0 && n > 0 && batch > 0;
  const int64_t rows_a = l3_is_n(transa) ? m : k, rows_b = l3_is_n(transb) ? k : n;
  if (nonempty && !scale_only && !A) return -7;
  if (lda < (rows_a > 1 ? rows_a : 1)) return -8;
  if (stride_a < 0) return -9;
  if (nonempty && !scale_only && !B) return -10;
  if (ldb < (rows_b > 1 ? rows_b : 1)) return -11;
  if (stride_b < 0) return -12;
  if (nonempty && !C) return -14;
  if (ldc < (m > 1 ? m : 1)) return -15;
  if (batch < 0) return -17;
  if (batch > 1 && n > 0 && stride_c < ldc * (n - 1) + m) return -16;  // the results must not overlap
  if (!nonempty) return B2_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (scale_only && beta == T(1)) return B2_OK;
  // grid.y carries at most 65535 problems per launch
  for (int64_t b0 = 0; b0 < batch; b0 += 65535) {
    const int nb = (int)((batch - b0) < 65535 ? (batch - b0) : 65535);
    T* Cb = C + b0 * stride_c;
    if (scale_only) {
      batch_scale_kernel<T><<<dim3(blocks_for(m * n), (unsigned)nb, 1), 256, 0, st>>>(m, n, beta, Cb, ldc, stride_c);
      if (cudaGetLastError() != cudaSuccess) return B2_ERR_LAUNCH;
      continue;
    }
    GemmExtra ex;
    ex.batch = nb, ex.stride_a = stride_a, ex.stride_b = stride_b, ex.stride_c = stride_c;
    const int rc = gemm_launch_checked<T>(B2_VARIANT_AUTO, l3_is_t(transa), l3_is_t(transb), m, n, k, alpha,
                                          A + b0 * stride_a, lda, B + b0 * stride_b, ldb, beta, Cb, ldc, ex, st);
    if (rc) return rc;
  }
  return B2_OK;
}

// ---- split-K: k cut into contiguous chunks, one partial product per chunk, summed in a fixed order ---------
// For small m*n and large k one CTA per C tile leaves most SMs idle; the chunks run as the batch dimension of
// one launch (A and B advance by one chunk per batch index, partial products go to workspace planes) and a
// second kernel forms C = alpha*(P_0 + P_1 + ...) + beta*C with the planes added in ascending order, so the
// result does not depend on scheduling.
template <typename T>
__global__ void splitk_reduce_kernel(int64_t m, int64_t n, int planes, const T* __restrict__ P, int64_t ldp,
                                     int64_t plane_stride, T alpha, T beta, T* __restrict__ C, int64_t ldc) {
  const int64_t total = m * n;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = idx % m, c = idx / m;
    const T* p = P + r + c * ldp;
    T acc = p[0];
    for (int s = 1; s < planes; ++s) acc += p[s * plane_stride];
    T* dst = C + r + c * ldc;
    *dst = (beta == T(0)) ? alpha * acc : alpha * acc + beta * *dst;
  }
}

constexpr int kSplitChunkUnit = 16;  // chunks are whole k-slabs, which also keeps every chunk 16-byte aligned

template <typename T>
int64_t splitk_pitch(int64_t m) {
  const int64_t vec = 16 / (int64_t)sizeof(T);
  return m < 1 ? vec : (m + vec - 1) / vec * vec;
}

int splitk_auto(int64_t m, int64_t n, int64_t k) {
  if (m <= 0 || n <= 0 || k <= 0) return 1;
  const int64_t tiles = ((m + 63) / 64) * ((n + 63) / 64);
  const int64_t slots = (int64_t)sm_count_cached() * 4;  // resident 64 x 64 tiles
  int64_t s = slots / tiles;
  if (s > k / 256) s = k / 256;  // every chunk at least 256 deep
  if (s > 64) s = 64;
  return s < 1 ? 1 : (int)s;
}

template <typename T>
int gemm_splitk(char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A, int64_t lda,
                const T* B, int64_t ldb, T beta, T* C, int64_t ldc, int splits, void* workspace,
                size_t workspace_bytes, void* cuda_stream) {
  const bool scale_only = (alpha == T(0) || k == 0);
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  if (splits < 0) return -14;
  if (splits == 0) splits = splitk_auto(m, n, k);
  if (splits > k) splits = k > 0 ? (int)k : 1;
  if (splits > 65535) splits = 65535;  // the chunks are the second grid dimension of one launch
  if (scale_only || splits <= 1 || m == 0 || n == 0)
    return gemm_entry<T>(B2_VARIANT_AUTO, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cuda_stream);
  const int64_t chunk = ((k + splits - 1) / splits + kSplitChunkUnit - 1) / kSplitChunkUnit * kSplitChunkUnit;
  const int64_t full = k / chunk, rest = k - full * chunk;
  const int planes = (int)(full + (rest > 0 ? 1 : 0));
  const int64_t ldp = splitk_pitch<T>(m), plane_stride = ldp * n;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 ||
      workspace_bytes < (size_t)planes * (size_t)plane_stride * sizeof(T))
    return B2_ERR_WORKSPACE;
  T* P = static_cast<T*>(workspace);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool ta = l3_is_t(transa), tb = l3_is_t(transb);
  const int64_t step_a = ta ? chunk : chunk * lda, step_b = tb ? chunk * ldb : chunk;  // one chunk further along k
  if (full > 0) {
    GemmExtra ex;
    ex.batch = (int)full, ex.stride_a = step_a, ex.stride_b = step_b, ex.stride_c = plane_stride;
    const int rc = gemm_launch_checked<T>(B2_VARIANT_AUTO, ta, tb, m, n, chunk, T(1), A, lda, B, ldb, T(0), P, ldp, ex, st);
    if (rc) return rc;
  }
  if (rest > 0) {
    const int rc = gemm_launch_checked<T>(B2_VARIANT_AUTO, ta, tb, m, n, rest, T(1), A + full * step_a, lda,
                                          B + full * step_b, ldb, T(0), P + full * plane_stride, ldp, GemmExtra(), st);
    if (rc) return rc;
  }
  splitk_reduce_kernel<T><<<blocks_for(m * n), 256, 0, st>>>(m, n, planes, P, ldp, plane_stride, alpha, beta, C, ldc);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

template <typename T>
size_t splitk_workspace_bytes(int64_t m, int64_t n, int64_t k, int splits) {
  if (m <= 0 || n <= 0 || k <= 0 || splits < 0) return 0;
  if (splits == 0) splits = splitk_auto(m, n, k);
  if (splits > k) splits = (int)k;
  if (splits > 65535) splits = 65535;
  if (splits <= 1) return 0;
  return (size_t)splits * (size_t)splitk_pitch<T>(m) * (size_t)n * sizeof(T);
}

}  // namespace
}  // namespace b2

extern "C" int b2_dsyrk(char uplo, char trans, int64_t n, int64_t k, double alpha, const double* A, int64_t lda,
                        double beta, double* C, int64_t ldc, void* cuda_stream) {
  return b2::syrk<double>(uplo, trans, n, k, alpha, A, lda, beta, C, ldc, cuda_stream);
}
extern "C" int b2_ssyrk(char uplo, char trans, int64_t n, int64_t k, float alpha, const float* A, int64_t lda,
                        float beta, float* C, int64_t ldc, void* cuda_stream) {
  return b2::syrk<float>(uplo, trans, n, k, alpha, A, lda, beta, C, ldc, cuda_stream);
}
extern "C" int b2_dgemm_strided_batched(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha,
                                        const double* A, int64_t lda, int64_t stride_a, const double* B, int64_t ldb,
                                        int64_t stride_b, double beta, double* C, int64_t ldc, int64_t stride_c,
                                        int64_t batch, void* cuda_stream) {
  return b2::gemm_strided_batched<double>(transa, transb, m, n, k, alpha, A, lda, stride_a, B, ldb, stride_b, beta, C,
                                          ldc, stride_c, batch, cuda_stream);
}
extern "C" int b2_sgemm_strided_batched(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha,
                                        const float* A, int64_t lda, int64_t stride_a, const float* B, int64_t ldb,
                                        int64_t stride_b, float beta, float* C, int64_t ldc, int64_t stride_c,
                                        int64_t batch, void* cuda_stream) {
  return b2::gemm_strided_batched<float>(transa, transb, m, n, k, alpha, A, lda, stride_a, B, ldb, stride_b, beta, C,
                                         ldc, stride_c, batch, cuda_stream);
}

extern "C" int b2_gemm_splitk_auto(int64_t m, int64_t n, int64_t k) { return b2::splitk_auto(m, n, k); }
extern "C" size_t b2_gemm_splitk_workspace_bytes(int dtype, int64_t m, int64_t n, int64_t k, int splits) {
  return dtype == 0 ? b2::splitk_workspace_bytes<double>(m, n, k, splits)
                    : b2::splitk_workspace_bytes<float>(m, n, k, splits);
}
extern "C" int b2_dgemm_splitk(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                               int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                               int splits, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::gemm_splitk<double>(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, splits, workspace,
                                 workspace_bytes, cuda_stream);
}
extern "C" int b2_sgemm_splitk(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                               int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc, int splits,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::gemm_splitk<float>(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, splits, workspace,
                                workspace_bytes, cuda_stream);
}
