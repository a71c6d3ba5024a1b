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
#include "gemm_kernel.cuh"

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

// Instruction-mix probes: the inner loop of a GEMM micro-kernel exactly as the GEMM kernels run it (the same
// compute() the kernels call: per k the shared-memory fragment loads plus the multiply-adds of one rank-1 update)
// over slabs that sit in shared memory from the start.  No global traffic, no staging code; BARRIER adds the one
// CTA-wide barrier per slab that the cp.async-staged kernels pass.  What such a probe reaches is the ceiling of the
// micro-kernel's instruction mix at the given residency; the gap between it and the full kernel is staging.
constexpr int kMixStages = 2;  // the slab address changes every round, so no load can be hoisted out of the loop

template <class Micro, bool BARRIER>
__global__ void __launch_bounds__(Micro::NT) probe_mix(long long iters, float* sink, long long* cycles) {
  using T = typename Micro::T;
  constexpr int STAGES = kMixStages;
  extern __shared__ __align__(16) unsigned char mix_smem[];
  T* sA = reinterpret_cast<T*>(mix_smem);
  T* sB = sA + STAGES * Micro::A_STAGE;
  for (int i = threadIdx.x; i < STAGES * Micro::A_STAGE; i += Micro::NT) sA[i] = T(1) + T(1e-3) * T(i % 61);
  for (int i = threadIdx.x; i < STAGES * Micro::B_STAGE; i += Micro::NT) sB[i] = T(1e-3) * T(1 + i % 53);
  __syncthreads();
  constexpr int WARPS_M = Micro::BM / Micro::WTM;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warp_m = warp % WARPS_M, warp_n = warp / WARPS_M;
  typename Micro::Acc acc;
  Micro::zero(acc);
  long long t0 = clock64();
  for (long long it = 0; it < iters; ++it) {
    const int st = (int)(it & (STAGES - 1));
    Micro::compute(acc, sA + st * Micro::A_STAGE, sB + st * Micro::B_STAGE, warp_m, warp_n, lane);
    if (BARRIER) __syncthreads();
  }
  long long t1 = clock64();
  const T s = Micro::checksum(acc);
  if (s == T(-1)) sink[0] = (float)s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

using MixFfma2_8x8 = b2::SimtMicro<float, 128, 64, 16, 2, 2, false, false, true, 8, 8>;
using MixFfma2_16x8 = b2::SimtMicro<float, 128, 128, 16, 1, 4, false, false, true, 16, 8>;
using MixDmma_64x64 = b2::DmmaMicro<64, 64, 16, 2, 2, false, false>;
using MixFfma_8x8 = b2::SimtMicro<float, 128, 64, 16, 2, 2, false, false, false, 8, 8>;
using MixFfma2_4x4 = b2::SimtMicro<float, 32, 32, 16, 1, 2, false, false, true, 4, 4>;
using MixDfma_8x8 = b2::SimtMicro<double, 128, 64, 16, 2, 2, false, false, false, 8, 8>;

// Shared memory that nothing touches, behind the slabs, pads each CTA so that exactly ceil(ctas / SMs) of them fit an SM: the
// probe then runs at the residency the caller asked for, evenly over the SMs, instead of wherever the block
// scheduler would pack CTAs this small.
template <class Micro, bool BARRIER>
int launch_mix_padded(int ctas, long long iters, void* sink, long long* cyc, cudaStream_t st) {
  int dev = 0, sms = 0, smem_sm = 0, reserved = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return B2_ERR_LAUNCH;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
  cudaDeviceGetAttribute(&reserved, cudaDevAttrReservedSharedMemoryPerBlock, dev);
  int optin = 0;
  cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  const long long slabs = (long long)kMixStages * (Micro::A_STAGE + Micro::B_STAGE) * sizeof(typename Micro::T);
  const int per_sm = (ctas + sms - 1) / sms;
  long long pad = ((long long)smem_sm / per_sm - reserved) / 1024 * 1024;  // slabs first, untouched padding behind
  if (pad < slabs) pad = slabs;
  if (pad > optin) pad = optin;
  if (cudaFuncSetAttribute(probe_mix<Micro, BARRIER>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pad) !=
      cudaSuccess)
    return B2_ERR_LAUNCH;
  // ask for the largest shared-memory carve-out, or the padded CTAs may not all fit beside the L1
  cudaFuncSetAttribute(probe_mix<Micro, BARRIER>, cudaFuncAttributePreferredSharedMemoryCarveout,
                       cudaSharedmemCarveoutMaxShared);
  probe_mix<Micro, BARRIER><<<ctas, Micro::NT, (size_t)pad, st>>>(iters, (float*)sink, cyc);
  return 0;
}

template <class Micro>
int launch_mix(bool barrier, int threads_per_cta, int ctas, long long iters, void* sink, long long* cyc,
               double* fma_per_thread_iter, cudaStream_t st) {
  if (threads_per_cta != Micro::NT) return -2;
  *fma_per_thread_iter = (double)Micro::BM * Micro::BN * Micro::BK / Micro::NT;
  return barrier ? launch_mix_padded<Micro, true>(ctas, iters, sink, cyc, st)
                 : launch_mix_padded<Micro, false>(ctas, iters, sink, cyc, st);
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
  const bool barrier = (kind & B2_PROBE_WITH_BARRIER) != 0;
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
    case B2_PROBE_MIX_FFMA2_8X8:
    case B2_PROBE_MIX_FFMA2_8X8 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixFfma2_8x8>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    case B2_PROBE_MIX_FFMA2_16X8:
    case B2_PROBE_MIX_FFMA2_16X8 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixFfma2_16x8>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    case B2_PROBE_MIX_DMMA_64X64:
    case B2_PROBE_MIX_DMMA_64X64 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixDmma_64x64>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    case B2_PROBE_MIX_FFMA_8X8:
    case B2_PROBE_MIX_FFMA_8X8 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixFfma_8x8>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    case B2_PROBE_MIX_FFMA2_4X4:
    case B2_PROBE_MIX_FFMA2_4X4 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixFfma2_4x4>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    case B2_PROBE_MIX_DFMA_8X8:
    case B2_PROBE_MIX_DFMA_8X8 | B2_PROBE_WITH_BARRIER:
      if (int rc = launch_mix<MixDfma_8x8>(barrier, threads_per_cta, ctas, iters, sink, cyc, fma_per_thread_iter, st))
        return rc;
      break;
    default:
      return -1;
  }
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}
