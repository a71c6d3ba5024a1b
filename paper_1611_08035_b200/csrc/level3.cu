// Level-3 routines built on the GEMM kernel (the paper's Abstract and Introduction name the level-3 BLAS as
// its consumers): the symmetric rank-k update, which is a GEMM with op(B) = op(A)^T restricted to one triangle of
// C, and the strided-batched GEMM, which is the GEMM grid replicated along grid.y.
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
  if (b > 148 * 16) b = 148 * 16;
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
