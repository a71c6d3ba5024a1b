// Register-resident throughput probes for the arithmetic pipes the GEMM micro-kernels use.
//
// The paper sizes a micro-kernel from per-pipeline throughputs (Section 4, "Estimating
// throughput": outer products per cycle = min over pipelines of rate / jobs).  On an SM the
// pipelines that matter are the FP64 FMA pipe, the FP64 tensor (DMMA) pipe and the FP32 FMA
// pipe; these probes measure their steady-state rates so the tile derivation uses measured
// numbers instead of remembered ones.  Every probe keeps all operands in registers, issues a
// long stream of independent multiply-adds and stores one value at the end so that nothing is
// optimised away.
#include <cuda_runtime.h>
#include <stdint.h>

#include "b2gemm.h"

namespace {

constexpr int kAcc = 32;  // independent accumulators per thread (FMA probes)

__global__ void probe_dfma(long long iters, double* sink, long long* cycles) {
  double acc[kAcc];
  const double a = 1.0 + 1e-9 * threadIdx.x, b = 1e-12;
#pragma unroll
  for (int i = 0; i < kAcc; ++i) acc[i] = 1.0 + i;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < kAcc; ++i) asm volatile("fma.rn.f64 %0, %0, %1, %2;" : "+d"(acc[i]) : "d"(a), "d"(b));
  }
  long long t1 = clock64();
  double s = 0;
#pragma unroll
  for (int i = 0; i < kAcc; ++i) s += acc[i];
  if (s == 123.456) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

__global__ void probe_ffma(long long iters, float* sink, long long* cycles) {
  float acc[kAcc];
  const float a = 1.0f + 1e-6f * threadIdx.x, b = 1e-9f;
#pragma unroll
  for (int i = 0; i < kAcc; ++i) acc[i] = 1.0f + i;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < kAcc; ++i) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(acc[i]) : "f"(a), "f"(b));
  }
  long long t1 = clock64();
  float s = 0;
#pragma unroll
  for (int i = 0; i < kAcc; ++i) s += acc[i];
  if (s == 123.456f) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// Packed FP32 pair FMA (fma.rn.f32x2, sm_100+): two IEEE fp32 multiply-adds per thread per instruction.
__global__ void probe_ffma2(long long iters, float* sink, long long* cycles) {
  unsigned long long acc[kAcc / 2];
  unsigned long long a, b;
  const float af = 1.0f + 1e-6f * threadIdx.x, bf = 1e-9f;
  asm volatile("mov.b64 %0, {%1, %1};" : "=l"(a) : "f"(af));
  asm volatile("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(bf));
#pragma unroll
  for (int i = 0; i < kAcc / 2; ++i) {
    const float v = 1.0f + i;
    asm volatile("mov.b64 %0, {%1, %1};" : "=l"(acc[i]) : "f"(v));
  }
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < kAcc / 2; ++i) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(acc[i]) : "l"(a), "l"(b));
  }
  long long t1 = clock64();
  float s = 0;
#pragma unroll
  for (int i = 0; i < kAcc / 2; ++i) {
    float lo, hi;
    asm volatile("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc[i]));
    s += lo + hi;
  }
  if (s == 123.456f) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// DMMA probes: NSETS independent accumulator fragments per warp, A/B fragments fixed.
template <int NSETS>
__global__ void probe_dmma_m8n8k4(long long iters, double* sink, long long* cycles) {
  double c[NSETS][2];
  const double a = 1e-3 * (threadIdx.x & 7), b = 1e-3 * (threadIdx.x & 3);
#pragma unroll
  for (int s = 0; s < NSETS; ++s) c[s][0] = c[s][1] = s;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int s = 0; s < NSETS; ++s)
      asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                   : "+d"(c[s][0]), "+d"(c[s][1]) : "d"(a), "d"(b));
  }
  long long t1 = clock64();
  double s = 0;
#pragma unroll
  for (int i = 0; i < NSETS; ++i) s += c[i][0] + c[i][1];
  if (s == 123.456) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int NSETS>
__global__ void probe_dmma_m16n8k4(long long iters, double* sink, long long* cycles) {
  double c[NSETS][4];
  const double a0 = 1e-3 * (threadIdx.x & 7), a1 = 2e-3, b = 1e-3 * (threadIdx.x & 3);
#pragma unroll
  for (int s = 0; s < NSETS; ++s) c[s][0] = c[s][1] = c[s][2] = c[s][3] = s;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int s = 0; s < NSETS; ++s)
      asm volatile("mma.sync.aligned.m16n8k4.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                   : "+d"(c[s][0]), "+d"(c[s][1]), "+d"(c[s][2]), "+d"(c[s][3]) : "d"(a0), "d"(a1), "d"(b));
  }
  long long t1 = clock64();
  double s = 0;
#pragma unroll
  for (int i = 0; i < NSETS; ++i) s += c[i][0] + c[i][1] + c[i][2] + c[i][3];
  if (s == 123.456) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int NSETS>
__global__ void probe_dmma_m16n8k8(long long iters, double* sink, long long* cycles) {
  double c[NSETS][4];
  const double a0 = 1e-3 * (threadIdx.x & 7), a1 = 2e-3, a2 = 3e-3, a3 = 4e-3;
  const double b0 = 1e-3 * (threadIdx.x & 3), b1 = 5e-3;
#pragma unroll
  for (int s = 0; s < NSETS; ++s) c[s][0] = c[s][1] = c[s][2] = c[s][3] = s;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int s = 0; s < NSETS; ++s)
      asm volatile("mma.sync.aligned.m16n8k8.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                   : "+d"(c[s][0]), "+d"(c[s][1]), "+d"(c[s][2]), "+d"(c[s][3])
                   : "d"(a0), "d"(a1), "d"(a2), "d"(a3), "d"(b0), "d"(b1));
  }
  long long t1 = clock64();
  double s = 0;
#pragma unroll
  for (int i = 0; i < NSETS; ++i) s += c[i][0] + c[i][1] + c[i][2] + c[i][3];
  if (s == 123.456) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int NSETS>
__global__ void probe_dmma_m16n8k16(long long iters, double* sink, long long* cycles) {
  double c[NSETS][4];
  double a[8], b[4];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = 1e-3 * (i + (threadIdx.x & 7));
#pragma unroll
  for (int i = 0; i < 4; ++i) b[i] = 1e-3 * (i + (threadIdx.x & 3));
#pragma unroll
  for (int s = 0; s < NSETS; ++s) c[s][0] = c[s][1] = c[s][2] = c[s][3] = s;
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
#pragma unroll
    for (int s = 0; s < NSETS; ++s)
      asm volatile(
          "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
          "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
          : "+d"(c[s][0]), "+d"(c[s][1]), "+d"(c[s][2]), "+d"(c[s][3])
          : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(a[4]), "d"(a[5]), "d"(a[6]), "d"(a[7]), "d"(b[0]),
            "d"(b[1]), "d"(b[2]), "d"(b[3]));
  }
  long long t1 = clock64();
  double s = 0;
#pragma unroll
  for (int i = 0; i < NSETS; ++i) s += c[i][0] + c[i][1] + c[i][2] + c[i][3];
  if (s == 123.456) sink[0] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace

extern "C" int b2_pipe_probe(int kind, int threads_per_cta, int ctas, int64_t iters, void* scratch,
                             size_t scratch_bytes, double* fma_per_thread_iter, void* cuda_stream) {
  if (threads_per_cta <= 0 || threads_per_cta > 1024 || (threads_per_cta % 32) != 0) return -2;
  if (ctas <= 0) return -3;
  if (iters <= 0) return -4;
  if (!scratch) return -5;
  if (scratch_bytes < 64 + sizeof(long long) * (size_t)ctas) return -6;
  if (!fma_per_thread_iter) return -7;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  double* sink = (double*)scratch;
  long long* cyc = (long long*)((char*)scratch + 64);
  constexpr int NS = 8;
  switch (kind) {
    case B2_PROBE_DFMA:
      probe_dfma<<<ctas, threads_per_cta, 0, st>>>(iters, sink, cyc);
      *fma_per_thread_iter = kAcc;
      break;
    case B2_PROBE_FFMA:
      probe_ffma<<<ctas, threads_per_cta, 0, st>>>(iters, (float*)sink, cyc);
      *fma_per_thread_iter = kAcc;
      break;
    case B2_PROBE_FFMA2:
      probe_ffma2<<<ctas, threads_per_cta, 0, st>>>(iters, (float*)sink, cyc);
      *fma_per_thread_iter = kAcc;
      break;
    case B2_PROBE_DMMA_M8N8K4:
      probe_dmma_m8n8k4<NS><<<ctas, threads_per_cta, 0, st>>>(iters, sink, cyc);
      *fma_per_thread_iter = NS * 8.0 * 8 * 4 / 32;
      break;
    case B2_PROBE_DMMA_M16N8K4:
      probe_dmma_m16n8k4<NS><<<ctas, threads_per_cta, 0, st>>>(iters, sink, cyc);
      *fma_per_thread_iter = NS * 16.0 * 8 * 4 / 32;
      break;
    case B2_PROBE_DMMA_M16N8K8:
      probe_dmma_m16n8k8<NS><<<ctas, threads_per_cta, 0, st>>>(iters, sink, cyc);
      *fma_per_thread_iter = NS * 16.0 * 8 * 8 / 32;
      break;
    case B2_PROBE_DMMA_M16N8K16:
      probe_dmma_m16n8k16<NS><<<ctas, threads_per_cta, 0, st>>>(iters, sink, cyc);
      *fma_per_thread_iter = NS * 16.0 * 8 * 16 / 32;
      break;
    default:
      return -1;
  }
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}
