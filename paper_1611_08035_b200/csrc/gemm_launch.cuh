// Host-side launch of one kernel variant: picks the (transA, transB, aligned) instantiation,
// raises the dynamic shared-memory limit once per device and launches on the caller's stream.
#pragma once
#include <atomic>

#include "b2gemm.h"
#include "gemm_kernel.cuh"

namespace b2 {

// Static description of a variant, used by the selector and by b2_gemm_query_config.
struct VariantInfo {
  const char* name;
  const char* micro;  // "dmma" | "dfma" | "ffma"
  int bm, bn, bk, stages, threads, ctas_per_sm;
  double efficiency;  // measured steady-state fraction of the arithmetic pipe's peak (large interior problems)
  int tm = 8, tn = 8;  // FMA micro-kernels: accumulator block per thread
  double per_tile_extra_clks = 0.0;  // ramp-up and epilogue time of a tile that its co-resident CTAs do not cover
  double transpose_b_cost = 7.0;     // FMA micro-kernels: loss to the transposing copy of a k-contiguous B is cost/BM
  bool can_ksplit = false;           // the kernel can split the k-loop of a tile over a thread-block cluster
};

template <typename T>
using LaunchFn = int (*)(const GemmArgs<T>& args, bool ta, bool tb, bool aligned, cudaStream_t stream);

template <class Kernel, int MIN_CTAS>
int launch_one(const GemmArgs<typename Kernel::T>& args, cudaStream_t stream) {
  // one flag per device; threads that get here together both set the (idempotent) attribute
  static std::atomic<bool> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return B2_ERR_LAUNCH;
  auto kfn = gemm_kernel<Kernel, MIN_CTAS>;
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Kernel::SMEM_BYTES) !=
        cudaSuccess)
      return B2_ERR_LAUNCH;
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  const long long tiles = (long long)args.tiles_m * args.tiles_n;
  if (tiles <= 0 || tiles > 0x7fffffffLL) return B2_ERR_LAUNCH;
  const int batch = args.batch > 0 ? args.batch : 1;
  if (args.ksplit > 1) {
    // k split: grid.z = cluster size; the CTAs (tile, problem, 0 .. ksplit-1) form one cluster
    if (!Kernel::KSPLIT_OK || args.ksplit > 8 || args.tri != 0) return B2_ERR_VARIANT;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tiles, (unsigned)batch, (unsigned)args.ksplit);
    cfg.blockDim = dim3(Kernel::NT, 1, 1);
    cfg.dynamicSmemBytes = Kernel::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = (unsigned)args.ksplit;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kfn, args) == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }
  kfn<<<dim3((unsigned)tiles, (unsigned)batch, 1), Kernel::NT, Kernel::SMEM_BYTES, stream>>>(args);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

// MicroT<TA, TB> is the micro-kernel policy for a transpose combination.
template <template <bool, bool> class MicroT, int STAGES, int MIN_CTAS>
struct VariantLauncher {
  template <bool TA, bool TB>
  using Micro = MicroT<TA, TB>;
  using T = typename MicroT<false, false>::T;

  template <bool TA, bool TB>
  static int pick_aligned(const GemmArgs<T>& a, bool aligned, cudaStream_t s) {
    if (aligned) return launch_one<GemmKernel<MicroT<TA, TB>, STAGES, TA, TB, true>, MIN_CTAS>(a, s);
    return launch_one<GemmKernel<MicroT<TA, TB>, STAGES, TA, TB, false>, MIN_CTAS>(a, s);
  }

  static int launch(const GemmArgs<T>& args_in, bool ta, bool tb, bool aligned, cudaStream_t s) {
    GemmArgs<T> a = args_in;
    constexpr int BM = MicroT<false, false>::BM, BN = MicroT<false, false>::BN;
    a.tiles_m = (int)((a.m + BM - 1) / BM);
    a.tiles_n = (int)((a.n + BN - 1) / BN);
    if (a.group_m <= 0) a.group_m = 8;
    if (!ta && !tb) return pick_aligned<false, false>(a, aligned, s);
    if (!ta && tb) return pick_aligned<false, true>(a, aligned, s);
    if (ta && !tb) return pick_aligned<true, false>(a, aligned, s);
    return pick_aligned<true, true>(a, aligned, s);
  }
};

// Variant tables, defined in gemm_f64_*.cu / gemm_f32_*.cu
int f64_variant_count();
const VariantInfo& f64_variant_info(int v);
LaunchFn<double> f64_variant_launch(int v);
int f32_variant_count();
const VariantInfo& f32_variant_info(int v);
LaunchFn<float> f32_variant_launch(int v);

}  // namespace b2
