// Complex double GEMM assembled from four launches of the real kernel (4M), or three (3M).
//
// The paper treats complex GEMM only as a consumer of the real kernel (Abstract); the
// decomposition used here is the textbook one on split real/imaginary planes:
//     A' = alpha*A (complex, elementwise),
//     Cr = A'r*Br - A'i*Bi + (beta*C)r,      Ci = A'r*Bi + A'i*Br + (beta*C)i.
// Steps: split kernels write the six planes into the caller's workspace, four real GEMMs
// accumulate into the two C planes, a merge kernel interleaves them back into C.
#include <atomic>

#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

// The element-wise kernels below run on a 2-D grid: blockIdx.x walks down a column in steps of the block size,
// blockIdx.y (with a stride loop, the grid's second extent is limited) over columns; no integer division per element.

// planes[0] = alpha_r*re - alpha_i*im, planes[1] = alpha_r*im + alpha_i*re of a rows x cols
// interleaved complex matrix with leading dimension ld (complex elements); plane pitch ldp.
// conj: the element is conjugated first (a conjugate transpose = plain transpose of these planes).
// Ps != nullptr: also the plane of sums planes[0] + planes[1] (the third operand of 3M).
__global__ void zsplit_scale_kernel(int64_t rows, int64_t cols, const double2* __restrict__ X, int64_t ld, double sr,
                                    double si, bool conj, double* __restrict__ Pr, double* __restrict__ Pi,
                                    double* __restrict__ Ps, int64_t ldp) {
  const bool plain = (sr == 1.0 && si == 0.0);
  for (int64_t c = blockIdx.y; c < cols; c += gridDim.y) {
    const double2* x = X + c * ld;
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < rows; r += (int64_t)gridDim.x * blockDim.x) {
      double2 v = x[r];
      if (conj) v.y = -v.y;
      double pr = v.x, pi = v.y;
      if (!plain) {
        pr = sr * v.x - si * v.y;
        pi = sr * v.y + si * v.x;
      }
      Pr[r + c * ldp] = pr;
      Pi[r + c * ldp] = pi;
      if (Ps) Ps[r + c * ldp] = pr + pi;
    }
  }
}

__global__ void zmerge_kernel(int64_t rows, int64_t cols, const double* __restrict__ Pr,
                              const double* __restrict__ Pi, int64_t ldp, double2* __restrict__ X, int64_t ld) {
  for (int64_t c = blockIdx.y; c < cols; c += gridDim.y)
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < rows; r += (int64_t)gridDim.x * blockDim.x)
      X[r + c * ld] = make_double2(Pr[r + c * ldp], Pi[r + c * ldp]);
}

// 3M: C := ((beta*C)r + T1 - T2,  ((beta*C)i - T1 - T2) + T3), the additions in exactly this order;
// beta == 0: C is not read.
__global__ void zmerge3m_kernel(int64_t rows, int64_t cols, const double* __restrict__ T1,
                                const double* __restrict__ T2, const double* __restrict__ T3, int64_t ldp, double br,
                                double bi, double2* __restrict__ X, int64_t ld) {
  const bool zero = (br == 0.0 && bi == 0.0);
  for (int64_t c = blockIdx.y; c < cols; c += gridDim.y) {
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < rows; r += (int64_t)gridDim.x * blockDim.x) {
      double cr = 0.0, ci = 0.0;
      if (!zero) {
        const double2 v = X[r + c * ld];
        cr = br * v.x - bi * v.y;
        ci = br * v.y + bi * v.x;
      }
      const double t1 = T1[r + c * ldp], t2 = T2[r + c * ldp], t3 = T3[r + c * ldp];
      X[r + c * ld] = make_double2((cr + t1) - t2, ((ci - t1) - t2) + t3);
    }
  }
}

// C := beta*C (complex); beta == 0 stores zeros without reading C.
__global__ void zscale_kernel(int64_t rows, int64_t cols, double br, double bi, double2* __restrict__ X, int64_t ld) {
  const bool zero = (br == 0.0 && bi == 0.0);
  for (int64_t c = blockIdx.y; c < cols; c += gridDim.y) {
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < rows; r += (int64_t)gridDim.x * blockDim.x) {
      double2* x = X + r + c * ld;
      if (zero) {
        *x = make_double2(0.0, 0.0);
      } else {
        const double2 v = *x;
        *x = make_double2(br * v.x - bi * v.y, br * v.y + bi * v.x);
      }
    }
  }
}

// grid for a rows x cols element-wise pass with 256-thread blocks
dim3 grid_for(int64_t rows, int64_t cols) {
  int64_t gx = (rows + 255) / 256;
  if (gx > 64) gx = 64;
  if (gx < 1) gx = 1;
  int64_t gy = cols < 1 ? 1 : (cols > 16384 ? 16384 : cols);
  return dim3((unsigned)gx, (unsigned)gy, 1);
}

struct Plan {
  int64_t ra, ca, rb, cb;     // stored rows/cols of A and B
  int64_t lpa, lpb, lpc;      // plane pitches (even, so plane columns are 16-byte aligned)
  size_t off[6], total;       // byte offsets of A'r, A'i, Br, Bi, Cr, Ci
  size_t sa, sb, sc;          // bytes of one plane of A, B, C
};

bool is_n(char c) { return c == 'N' || c == 'n'; }
bool is_t(char c) { return c == 'T' || c == 't'; }
bool is_c(char c) { return c == 'C' || c == 'c'; }
bool is_op(char c) { return is_n(c) || is_t(c) || is_c(c); }
char real_op(char c) { return is_n(c) ? 'N' : 'T'; }  // the transpose the real kernels see

Plan make_plan(char transa, char transb, int64_t m, int64_t n, int64_t k) {
  Plan p;
  p.ra = is_n(transa) ? m : k, p.ca = is_n(transa) ? k : m;
  p.rb = is_n(transb) ? k : n, p.cb = is_n(transb) ? n : k;
  auto even = [](int64_t x) { return x < 1 ? (int64_t)2 : (x + 1) / 2 * 2; };
  p.lpa = even(p.ra), p.lpb = even(p.rb), p.lpc = even(m);
  const size_t sa = round_up((size_t)p.lpa * (size_t)(p.ca > 0 ? p.ca : 0) * 8, 256);
  const size_t sb = round_up((size_t)p.lpb * (size_t)(p.cb > 0 ? p.cb : 0) * 8, 256);
  const size_t sc = round_up((size_t)p.lpc * (size_t)(n > 0 ? n : 0) * 8, 256);
  p.off[0] = 0, p.off[1] = sa, p.off[2] = 2 * sa, p.off[3] = 2 * sa + sb, p.off[4] = 2 * sa + 2 * sb;
  p.off[5] = p.off[4] + sc;
  p.total = p.off[5] + sc;
  p.sa = sa, p.sb = sb, p.sc = sc;
  return p;
}

}  // namespace
}  // namespace b2

extern "C" size_t b2_zgemm4m_workspace_bytes(char transa, char transb, int64_t m, int64_t n, int64_t k) {
  using namespace b2;
  if (!is_op(transa) || !is_op(transb) || m < 0 || n < 0 || k < 0) return 0;
  return make_plan(transa, transb, m, n, k).total;
}

namespace b2 {
namespace {
// Where the six planes of a 4M call live: the caller's workspace, or the array built into the library.
struct Scratch {
  void* workspace;
  size_t workspace_bytes;
  bool built_in;  // resolve the built-in array (after the argument checks and quick returns) instead
};
void* builtin_scratch();  // device address of the built-in array on the current device (nullptr on failure)

int zgemm4m_run(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2], const void* A,
                int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C, int64_t ldc, Scratch scratch,
                void* cuda_stream) {
  if (!is_op(transa)) return -1;
  if (!is_op(transb)) return -2;
  if (!alpha) return -6;
  if (!beta) return -11;
  const double ar = alpha[0], ai = alpha[1], br = beta[0], bi = beta[1];
  const bool alpha0 = (ar == 0.0 && ai == 0.0), beta0 = (br == 0.0 && bi == 0.0);
  const bool scale_only = alpha0 || k == 0;
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  if (m == 0 || n == 0) return B2_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  double2* Cz = static_cast<double2*>(C);
  if (scale_only) {
    if (br == 1.0 && bi == 0.0) return B2_OK;
    zscale_kernel<<<grid_for(m, n), 256, 0, st>>>(m, n, br, bi, Cz, ldc);
    return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }
  const Plan p = make_plan(transa, transb, m, n, k);
  void* workspace = scratch.workspace;
  if (scratch.built_in) {
    // only a call that really splits planes is held to the size of the built-in array
    if (p.total > (size_t)B2_ZGEMM4M_STATIC_BYTES) return B2_ERR_STATIC_LIMIT;
    workspace = builtin_scratch();
    if (!workspace) return B2_ERR_LAUNCH;
  } else if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 || scratch.workspace_bytes < p.total) {
    return B2_ERR_WORKSPACE;
  }
  char* w = static_cast<char*>(workspace);
  double* Apr = reinterpret_cast<double*>(w + p.off[0]);
  double* Api = reinterpret_cast<double*>(w + p.off[1]);
  double* Br = reinterpret_cast<double*>(w + p.off[2]);
  double* Bi = reinterpret_cast<double*>(w + p.off[3]);
  double* Cr = reinterpret_cast<double*>(w + p.off[4]);
  double* Ci = reinterpret_cast<double*>(w + p.off[5]);

  zsplit_scale_kernel<<<grid_for(p.ra, p.ca), 256, 0, st>>>(p.ra, p.ca, static_cast<const double2*>(A), lda, ar, ai,
                                                           is_c(transa), Apr, Api, nullptr, p.lpa);
  zsplit_scale_kernel<<<grid_for(p.rb, p.cb), 256, 0, st>>>(p.rb, p.cb, static_cast<const double2*>(B), ldb, 1.0,
                                                           0.0, is_c(transb), Br, Bi, nullptr, p.lpb);
  double first_beta = 0.0;
  if (!beta0) {
    zsplit_scale_kernel<<<grid_for(m, n), 256, 0, st>>>(m, n, Cz, ldc, br, bi, false, Cr, Ci, nullptr, p.lpc);
    first_beta = 1.0;
  }
  transa = real_op(transa), transb = real_op(transb);
  if (cudaGetLastError() != cudaSuccess) return B2_ERR_LAUNCH;
  int rc;
  // Cr = A'r*Br + (beta*C)r ; Cr -= A'i*Bi
  rc = gemm_entry<double>(B2_VARIANT_AUTO, transa, transb, m, n, k, 1.0, Apr, p.lpa, Br, p.lpb, first_beta, Cr, p.lpc, st);
  if (rc) return rc;
  rc = gemm_entry<double>(B2_VARIANT_AUTO, transa, transb, m, n, k, -1.0, Api, p.lpa, Bi, p.lpb, 1.0, Cr, p.lpc, st);
  if (rc) return rc;
  // Ci = A'r*Bi + (beta*C)i ; Ci += A'i*Br
  rc = gemm_entry<double>(B2_VARIANT_AUTO, transa, transb, m, n, k, 1.0, Apr, p.lpa, Bi, p.lpb, first_beta, Ci, p.lpc, st);
  if (rc) return rc;
  rc = gemm_entry<double>(B2_VARIANT_AUTO, transa, transb, m, n, k, 1.0, Api, p.lpa, Br, p.lpb, 1.0, Ci, p.lpc, st);
  if (rc) return rc;
  zmerge_kernel<<<grid_for(m, n), 256, 0, st>>>(m, n, Cr, Ci, p.lpc, Cz, ldc);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}
}  // namespace
}  // namespace b2

extern "C" int b2_zgemm4m(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2],
                          const void* A, int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C,
                          int64_t ldc, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::zgemm4m_run(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                         b2::Scratch{workspace, workspace_bytes, false}, cuda_stream);
}

// ---- 3M: three real products instead of four ----------------------------------------------------
// Planes in the workspace: A'r, A'i, A'r+A'i | Br, Bi, Br+Bi | T1, T2, T3 (m x n each).
extern "C" size_t b2_zgemm3m_workspace_bytes(char transa, char transb, int64_t m, int64_t n, int64_t k) {
  using namespace b2;
  if (!is_op(transa) || !is_op(transb) || m < 0 || n < 0 || k < 0) return 0;
  const Plan p = make_plan(transa, transb, m, n, k);
  return 3 * (p.sa + p.sb + p.sc);
}

extern "C" int b2_zgemm3m(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2],
                          const void* A, int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C,
                          int64_t ldc, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  using namespace b2;
  if (!is_op(transa)) return -1;
  if (!is_op(transb)) return -2;
  if (!alpha) return -6;
  if (!beta) return -11;
  const double ar = alpha[0], ai = alpha[1], br = beta[0], bi = beta[1];
  const bool alpha0 = (ar == 0.0 && ai == 0.0);
  const bool scale_only = alpha0 || k == 0;
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  if (m == 0 || n == 0) return B2_OK;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  double2* Cz = static_cast<double2*>(C);
  if (scale_only) {
    if (br == 1.0 && bi == 0.0) return B2_OK;
    zscale_kernel<<<grid_for(m, n), 256, 0, st>>>(m, n, br, bi, Cz, ldc);
    return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }
  const Plan p = make_plan(transa, transb, m, n, k);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 ||
      workspace_bytes < 3 * (p.sa + p.sb + p.sc))
    return B2_ERR_WORKSPACE;
  char* w = static_cast<char*>(workspace);
  double* Ap[3];
  double* Bp[3];
  double* T[3];
  for (int i = 0; i < 3; ++i) {
    Ap[i] = reinterpret_cast<double*>(w + i * p.sa);
    Bp[i] = reinterpret_cast<double*>(w + 3 * p.sa + i * p.sb);
    T[i] = reinterpret_cast<double*>(w + 3 * p.sa + 3 * p.sb + i * p.sc);
  }
  zsplit_scale_kernel<<<grid_for(p.ra, p.ca), 256, 0, st>>>(p.ra, p.ca, static_cast<const double2*>(A), lda, ar, ai,
                                                           is_c(transa), Ap[0], Ap[1], Ap[2], p.lpa);
  zsplit_scale_kernel<<<grid_for(p.rb, p.cb), 256, 0, st>>>(p.rb, p.cb, static_cast<const double2*>(B), ldb, 1.0,
                                                           0.0, is_c(transb), Bp[0], Bp[1], Bp[2], p.lpb);
  if (cudaGetLastError() != cudaSuccess) return B2_ERR_LAUNCH;
  const char ta = real_op(transa), tb = real_op(transb);
  for (int i = 0; i < 3; ++i) {  // T1 = A'r*Br, T2 = A'i*Bi, T3 = (A'r+A'i)*(Br+Bi)
    const int rc = gemm_entry<double>(B2_VARIANT_AUTO, ta, tb, m, n, k, 1.0, Ap[i], p.lpa, Bp[i], p.lpb, 0.0, T[i],
                                      p.lpc, st);
    if (rc) return rc;
  }
  zmerge3m_kernel<<<grid_for(m, n), 256, 0, st>>>(m, n, T[0], T[1], T[2], p.lpc, br, bi, Cz, ldc);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

// ---- b2_zgemm4m without a caller-provided workspace -------------------------------------------
// The scratch planes live in the library image.  In host code the array's name is only a
// host-side stand-in for the symbol, not a device address: the address each device maps it
// to is looked up once per device (with that device current) by cudaGetSymbolAddress and cached.
// Two host threads that make their first call on a device together both look the address up and
// store the same value (atomic slots), which is harmless.
static __device__ __align__(256) unsigned char g_zgemm4m_scratch[B2_ZGEMM4M_STATIC_BYTES];

namespace b2 {
namespace {
void* builtin_scratch() {
  static std::atomic<void*> by_device[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  void* ptr = by_device[dev].load(std::memory_order_acquire);
  if (!ptr) {
    if (cudaGetSymbolAddress(&ptr, g_zgemm4m_scratch) != cudaSuccess || !ptr) return nullptr;
    by_device[dev].store(ptr, std::memory_order_release);
  }
  return ptr;
}
}  // namespace
}  // namespace b2

extern "C" int b2_zgemm4m_static(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2],
                                 const void* A, int64_t lda, const void* B, int64_t ldb, const double beta[2],
                                 void* C, int64_t ldc, void* cuda_stream) {
  return b2::zgemm4m_run(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                         b2::Scratch{nullptr, 0, true}, cuda_stream);
}
