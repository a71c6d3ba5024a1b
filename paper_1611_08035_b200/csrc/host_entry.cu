// Host-buffer forms of the real GEMM: copy the referenced parts of A, B (and C when beta != 0)
// into the caller's device workspace, run the device entry point, copy the result back.
//
// Copies and multiplication are pipelined on a copy-in stream, the caller's stream and a copy-out stream (PCIe is
// full duplex), in one of two orders:
//   * column panels of C (small and medium problems): A goes up first, then the panels of B (and of C when
//     beta != 0) follow while the kernel works on the panels that have arrived and finished panels go back.
//     Each panel is one call of the device entry point: the same bits as b2_dgemm / b2_sgemm.  The time is the
//     upload of A plus about max(copy time, compute time).
//   * k-chunks first (large problems, k >= 2048): A's upload alone would leave the GPU idle for as long as a
//     third of the multiplication takes, so A and B go up chunk by chunk along k and the kernel adds
//     alpha * A_p * B_p to all of C as each chunk p arrives (beta = 0 for the first chunk, 1 afterwards); C's old
//     values travel last, into a buffer of their own; the last chunk runs column panel by column panel, each
//     followed by C_panel += beta * C_old_panel and its copy back.  Only the first chunk's upload and the last
//     panel's download are exposed.  The sum over k is formed chunk by chunk: the same error bound as the single
//     call, not the same rounding.
// The two helper streams and a few events are created on the first call on a device and kept (no device memory is
// allocated); calls are serialised by a mutex.
#include <mutex>

#include "b2gemm.h"
#include "entry.h"

namespace b2 {
namespace {

struct HostPlan {
  int64_t ra, ca, rb, cb, lda_d, ldb_d, ldc_d;
  size_t off_b, off_c, off_cold, total;
  bool by_k;  // k-chunks first
};

constexpr int64_t kChunkMinK = 2048;         // k-chunks pay from here on ...
constexpr int64_t kChunkMinMN = 1ll << 22;   // ... for at least this many elements of C
constexpr int kMaxChunks = 8;

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
  p.by_k = k >= kChunkMinK && m * n >= kChunkMinMN;
  p.off_b = sa, p.off_c = sa + sb, p.off_cold = sa + sb + sc;
  p.total = sa + sb + sc + (p.by_k ? sc : 0);  // by k: the old values of C wait in a buffer of their own
  return p;
}

// Helper streams and events of the pipelined host-buffer calls, one set per device, created on first use.
constexpr int kMaxPanels = 20;  // events per kind; the panel count itself is capped at 16 (+1 for a cut last panel)
struct HostPipe {
  cudaStream_t cin, cout;
  cudaEvent_t start, a_ready, out_done, in[kMaxPanels], done[kMaxPanels], old_in[kMaxPanels];
};

// C(:, 0:cols) += beta * Cold(:, 0:cols), both with leading dimension ld
template <typename T>
__global__ void add_scaled_kernel(int64_t rows, int64_t cols, T beta, T* C, const T* Cold, int64_t ld) {
  const int64_t total = rows * cols;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t at = (i / rows) * ld + i % rows;
    C[at] = C[at] + beta * Cold[at];
  }
}
HostPipe* host_pipe() {
  static HostPipe pipes[64];
  static bool ready[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ready[dev]) {
    HostPipe& h = pipes[dev];
    bool good = cudaStreamCreateWithFlags(&h.cin, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&h.cout, cudaStreamNonBlocking) == cudaSuccess;
    auto ev = [&good](cudaEvent_t* e) { good = good && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
    ev(&h.start), ev(&h.a_ready), ev(&h.out_done);
    for (int i = 0; i < kMaxPanels; ++i) ev(&h.in[i]), ev(&h.done[i]), ev(&h.old_in[i]);
    if (!good) return nullptr;
    ready[dev] = true;
  }
  return &pipes[dev];
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

  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe* hp = host_pipe();
  if (!hp) return B2_ERR_LAUNCH;
  auto ok = [](cudaError_t err) { return err == cudaSuccess; };

  // column panels of C: at least 512 columns each, at most kMaxPanels, multiples of 64 columns
  int64_t panels = n / 1024;
  panels = panels < 1 ? 1 : (panels > 16 ? 16 : panels);
  const int64_t width = ((n + panels - 1) / panels + 63) / 64 * 64;
  const bool tb = !h_is_n(transb);

  // both helper streams start after whatever the caller's stream has queued so far
  if (!ok(cudaEventRecord(hp->start, st)) || !ok(cudaStreamWaitEvent(hp->cin, hp->start, 0)) ||
      !ok(cudaStreamWaitEvent(hp->cout, hp->start, 0)))
    return B2_ERR_LAUNCH;
  if (p.by_k && !scale_only) {
    // ---- k-chunks first -------------------------------------------------------------------------------
    const bool ta = !h_is_n(transa);
    T* dCold = reinterpret_cast<T*>(w + p.off_cold);
    int64_t chunks = k / 1024;
    chunks = chunks < 2 ? 2 : (chunks > kMaxChunks ? kMaxChunks : chunks);
    const int64_t kc = ((k + chunks - 1) / chunks + 63) / 64 * 64;
    // The first chunks are added to all of C as they arrive; the last three eighths of k are applied column
    // panel by column panel, so that finished panels leave over about as long as the copy back of C takes
    // (a third of the multiplication on this machine) instead of all at the end.
    const int64_t nchunks = (k + kc - 1) / kc;
    int64_t late = (3 * nchunks + 4) / 8;
    late = late < 1 ? 1 : late;
    const int64_t k1 = (nchunks - late) * kc;  // first k of the part applied by panels
    // chunk boundaries; the first chunk is cut once more, a quarter first, so that the multiplication starts sooner
    int64_t kb[kMaxChunks + 3];
    int nb = 0;
    kb[nb++] = 0;
    const int64_t quarter = kc / 4 / 64 * 64;
    if (quarter >= 128) kb[nb++] = quarter;
    for (int64_t k0 = kc; k0 < k; k0 += kc) kb[nb++] = k0;
    kb[nb] = k;
    // column panels of the last part; the last panel is cut in two, so that less is left to copy back at the end
    int64_t jb[kMaxPanels + 1];
    int npanels = 0;
    for (int64_t j0 = 0; j0 < n; j0 += width) jb[npanels++] = j0;
    jb[npanels] = n;
    {
      const int64_t last = n - jb[npanels - 1], half = last / 2 / 64 * 64;
      if (half >= 128 && npanels < kMaxPanels) {
        jb[npanels + 1] = n;
        jb[npanels] = jb[npanels - 1] + half;
        ++npanels;
      }
    }
    for (int nc = 0; nc < nb; ++nc) {
      const int64_t k0 = kb[nc], kk = kb[nc + 1] - k0;
      // chunk of op(A): columns k0.. of an m x k matrix, or rows k0.. of a k x m one; of op(B) the other way round
      cudaError_t err =
          ta ? cudaMemcpy2DAsync(dA + k0, p.lda_d * e, A + k0, lda * e, kk * e, p.ca, cudaMemcpyHostToDevice, hp->cin)
             : cudaMemcpy2DAsync(dA + k0 * p.lda_d, p.lda_d * e, A + k0 * lda, lda * e, p.ra * e, kk,
                                 cudaMemcpyHostToDevice, hp->cin);
      if (!ok(err)) return B2_ERR_LAUNCH;
      err = tb ? cudaMemcpy2DAsync(dB + k0 * p.ldb_d, p.ldb_d * e, B + k0 * ldb, ldb * e, p.rb * e, kk,
                                   cudaMemcpyHostToDevice, hp->cin)
               : cudaMemcpy2DAsync(dB + k0, p.ldb_d * e, B + k0, ldb * e, kk * e, p.cb, cudaMemcpyHostToDevice, hp->cin);
      if (!ok(err)) return B2_ERR_LAUNCH;
      if (!ok(cudaEventRecord(hp->in[nc], hp->cin)) || !ok(cudaStreamWaitEvent(st, hp->in[nc], 0))) return B2_ERR_LAUNCH;
      if (k0 < k1) {
        const int rc = gemm_entry<T>(B2_VARIANT_AUTO, transa, transb, m, n, kk, alpha, ta ? dA + k0 : dA + k0 * p.lda_d,
                                     p.lda_d, tb ? dB + k0 * p.ldb_d : dB + k0, p.ldb_d, k0 == 0 ? T(0) : T(1), dC,
                                     p.ldc_d, cuda_stream);
        if (rc) return rc;
      }
    }
    // the old values of C follow A and B, panel by panel
    if (beta != T(0)) {
      for (int np = 0; np < npanels; ++np) {
        const int64_t j0 = jb[np], nj = jb[np + 1] - j0;
        if (!ok(cudaMemcpy2DAsync(dCold + j0 * p.ldc_d, p.ldc_d * e, C + j0 * ldc, ldc * e, m * e, nj,
                                  cudaMemcpyHostToDevice, hp->cin)) ||
            !ok(cudaEventRecord(hp->old_in[np], hp->cin)))
          return B2_ERR_LAUNCH;
      }
    }
    // the rest of k (all of A and B is on the device: the caller's stream has waited for every chunk)
    const T* dAk = ta ? dA + k1 : dA + k1 * p.lda_d;
    const T* dBk = tb ? dB + k1 * p.ldb_d : dB + k1;
    for (int np = 0; np < npanels; ++np) {
      const int64_t j0 = jb[np], nj = jb[np + 1] - j0;
      T* dCj = dC + j0 * p.ldc_d;
      const int rc = gemm_entry<T>(B2_VARIANT_AUTO, transa, transb, m, nj, k - k1, alpha, dAk, p.lda_d,
                                   tb ? dBk + j0 : dBk + j0 * p.ldb_d, p.ldb_d, k1 == 0 ? T(0) : T(1), dCj, p.ldc_d,
                                   cuda_stream);
      if (rc) return rc;
      if (beta != T(0)) {
        if (!ok(cudaStreamWaitEvent(st, hp->old_in[np], 0))) return B2_ERR_LAUNCH;
        const int64_t blocks = (m * nj + 255) / 256, cap = (int64_t)sm_count_cached() * 16;
        add_scaled_kernel<T><<<(unsigned)(blocks > cap ? cap : blocks), 256, 0, st>>>(m, nj, beta, dCj,
                                                                                   dCold + j0 * p.ldc_d, p.ldc_d);
        if (cudaGetLastError() != cudaSuccess) return B2_ERR_LAUNCH;
      }
      if (!ok(cudaEventRecord(hp->done[np], st)) || !ok(cudaStreamWaitEvent(hp->cout, hp->done[np], 0)) ||
          !ok(cudaMemcpy2DAsync(C + j0 * ldc, ldc * e, dCj, p.ldc_d * e, m * e, nj, cudaMemcpyDeviceToHost, hp->cout)))
        return B2_ERR_LAUNCH;
    }
    if (!ok(cudaEventRecord(hp->out_done, hp->cout)) || !ok(cudaStreamWaitEvent(st, hp->out_done, 0)))
      return B2_ERR_LAUNCH;
    return cudaStreamSynchronize(st) == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }

  // ---- column panels of C ---------------------------------------------------------------------------------
  if (!scale_only) {
    if (!ok(cudaMemcpy2DAsync(dA, p.lda_d * e, A, lda * e, p.ra * e, p.ca, cudaMemcpyHostToDevice, hp->cin)))
      return B2_ERR_LAUNCH;
  }
  if (!ok(cudaEventRecord(hp->a_ready, hp->cin)) || !ok(cudaStreamWaitEvent(st, hp->a_ready, 0))) return B2_ERR_LAUNCH;
  int np = 0;
  for (int64_t j0 = 0; j0 < n; j0 += width, ++np) {
    const int64_t nj = (n - j0) < width ? (n - j0) : width;
    if (!scale_only) {
      // panel of op(B): columns j0.. of a k x n matrix, or rows j0.. of an n x k matrix
      const cudaError_t err =
          tb ? cudaMemcpy2DAsync(dB + j0, p.ldb_d * e, B + j0, ldb * e, nj * e, p.cb, cudaMemcpyHostToDevice, hp->cin)
             : cudaMemcpy2DAsync(dB + j0 * p.ldb_d, p.ldb_d * e, B + j0 * ldb, ldb * e, p.rb * e, nj,
                                 cudaMemcpyHostToDevice, hp->cin);
      if (!ok(err)) return B2_ERR_LAUNCH;
    }
    if (beta != T(0)) {
      if (!ok(cudaMemcpy2DAsync(dC + j0 * p.ldc_d, p.ldc_d * e, C + j0 * ldc, ldc * e, m * e, nj, cudaMemcpyHostToDevice,
                                hp->cin)))
        return B2_ERR_LAUNCH;
    }
    if (!ok(cudaEventRecord(hp->in[np], hp->cin)) || !ok(cudaStreamWaitEvent(st, hp->in[np], 0))) return B2_ERR_LAUNCH;
    const T* dBj = tb ? dB + j0 : dB + j0 * p.ldb_d;
    const int rc = gemm_entry<T>(B2_VARIANT_AUTO, transa, transb, m, nj, k, alpha, dA, p.lda_d, dBj, p.ldb_d, beta,
                                 dC + j0 * p.ldc_d, p.ldc_d, cuda_stream);
    if (rc) return rc;
    if (!ok(cudaEventRecord(hp->done[np], st)) || !ok(cudaStreamWaitEvent(hp->cout, hp->done[np], 0)))
      return B2_ERR_LAUNCH;
    if (!ok(cudaMemcpy2DAsync(C + j0 * ldc, ldc * e, dC + j0 * p.ldc_d, p.ldc_d * e, m * e, nj, cudaMemcpyDeviceToHost,
                              hp->cout)))
      return B2_ERR_LAUNCH;
  }
  if (!ok(cudaEventRecord(hp->out_done, hp->cout)) || !ok(cudaStreamWaitEvent(st, hp->out_done, 0))) return B2_ERR_LAUNCH;
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
