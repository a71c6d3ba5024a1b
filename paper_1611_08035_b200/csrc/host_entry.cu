// Host-buffer forms of the real GEMM: copy the referenced parts of A, B (and C when beta != 0)
// into the caller's device workspace, run the device entry point, copy the result back.
#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

struct HostPlan {
  int64_t ra, ca, rb, cb, lda_d, ldb_d, ldc_d;
  size_t off_b, off_c, total;
};

bool h_is_n(char c) { return c == 'N' || c == 'n'; }

HostPlan host_plan(int elem, char transa, char transb, int64_t m, int64_t n, int64_t k) {
  HostPlan p;
  p.ra = h_is_n(transa) ? m : k, p.ca = h_is_n(transa) ? k : m;
  p.rb = h_is_n(transb) ? k : n, p.cb = h_is_n(transb) ? n : k;
  const int64_t vec = 16 / elem;
  auto pad = [vec](int64_t x) { return x < 1 ? vec : (x + vec - 1) / vec * vec; };
  p.lda_d = pad(p.ra), p.ldb_d = pad(p.rb), p.ldc_d = pad(m);
  const size_t sa = round_up((size_t)p.lda_d * (size_t)(p.ca > 0 ? p.ca : 0) * elem, 256);
  const size_t sb = round_up((size_t)p.ldb_d * (size_t)(p.cb > 0 ? p.cb : 0) * elem, 256);
  const size_t sc = round_up((size_t)p.ldc_d * (size_t)(n > 0 ? n : 0) * elem, 256);
  p.off_b = sa, p.off_c = sa + sb, p.total = sa + sb + sc;
  return p;
}

template <typename T>
int gemm_host(char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A, int64_t lda, const T* B,
              int64_t ldb, T beta, T* C, int64_t ldc, void* ws, size_t ws_bytes, void* cuda_stream) {
  const bool scale_only = (alpha == T(0) || k == 0);
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  if (m == 0 || n == 0) return B2_OK;
  if (scale_only && beta == T(1)) return B2_OK;
  const HostPlan p = host_plan((int)sizeof(T), transa, transb, m, n, k);
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < p.total) return B2_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* w = static_cast<char*>(ws);
  T* dA = reinterpret_cast<T*>(w);
  T* dB = reinterpret_cast<T*>(w + p.off_b);
  T* dC = reinterpret_cast<T*>(w + p.off_c);
  const size_t e = sizeof(T);
  if (!scale_only) {
    if (cudaMemcpy2DAsync(dA, p.lda_d * e, A, lda * e, p.ra * e, p.ca, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return B2_ERR_LAUNCH;
    if (cudaMemcpy2DAsync(dB, p.ldb_d * e, B, ldb * e, p.rb * e, p.cb, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return B2_ERR_LAUNCH;
  }
  if (beta != T(0)) {
    if (cudaMemcpy2DAsync(dC, p.ldc_d * e, C, ldc * e, m * e, n, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return B2_ERR_LAUNCH;
  }
  const int rc = gemm_entry<T>(B2_VARIANT_AUTO, transa, transb, m, n, k, alpha, dA, p.lda_d, dB, p.ldb_d, beta, dC,
                               p.ldc_d, cuda_stream);
  if (rc) return rc;
  if (cudaMemcpy2DAsync(C, ldc * e, dC, p.ldc_d * e, m * e, n, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return B2_ERR_LAUNCH;
  return cudaStreamSynchronize(st) == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

}  // namespace
}  // namespace b2

extern "C" size_t b2_gemm_host_workspace_bytes(int dtype, char transa, char transb, int64_t m, int64_t n, int64_t k) {
  if ((dtype != B2_F64 && dtype != B2_F32) || m < 0 || n < 0 || k < 0) return 0;
  return b2::host_plan(dtype == B2_F64 ? 8 : 4, transa, transb, m, n, k).total;
}

extern "C" int b2_dgemm_host(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                             int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                             void* dev_workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::gemm_host<double>(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, dev_workspace,
                               workspace_bytes, cuda_stream);
}

extern "C" int b2_sgemm_host(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                             int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                             void* dev_workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::gemm_host<float>(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, dev_workspace,
                              workspace_bytes, cuda_stream);
}
