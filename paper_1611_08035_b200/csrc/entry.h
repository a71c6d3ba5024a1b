// Internal declarations shared by the translation units that implement C-ABI entry points.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace b2 {

// Real GEMM behind b2_dgemm / b2_sgemm (argument check, quick returns, variant choice, launch).
template <typename T>
int gemm_entry(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A,
               int64_t lda, const T* B, int64_t ldb, T beta, T* C, int64_t ldc, void* cuda_stream);

// Extras of a launch beyond plain GEMM: triangular update (tri = 1 lower, 2 upper) and strided batches.
struct GemmExtra {
  int tri = 0;
  int batch = 1;
  int64_t stride_a = 0, stride_b = 0, stride_c = 0;
  int ksplit = 0;  // k split of every tile over a cluster: 0 = the selector's choice (automatic variant) or none
};
// Variant choice and launch of an already checked, non-trivial problem (m, n, k > 0, alpha != 0); ta/tb: transposed.
template <typename T>
int gemm_launch_checked(int variant, bool ta, bool tb, int64_t m, int64_t n, int64_t k, T alpha, const T* A,
                        int64_t lda, const T* B, int64_t ldb, T beta, T* C, int64_t ldc, const GemmExtra& ex,
                        cudaStream_t stream);

// BLAS argument check; 0 or the negative 1-based index of the first illegal argument.
int check_gemm_args(char transa, char transb, int64_t m, int64_t n, int64_t k, const void* A, int64_t lda,
                    const void* B, int64_t ldb, const void* C, int64_t ldc, bool reads_ab);

// Multiprocessor count of the current device (queried once per device; 148 when the query fails).
int sm_count_cached();

inline size_t round_up(size_t x, size_t to) { return (x + to - 1) / to * to; }

}  // namespace b2
