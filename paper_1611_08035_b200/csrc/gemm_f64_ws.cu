// fp64 DMMA kernels as persistent, warp-specialised CTAs (gemm_ws.cuh): tensor maps, launch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "b2gemm.h"
#include "entry.h"
#include "gemm_launch.cuh"
#include "gemm_ws.cuh"

namespace b2 {
namespace {

template <class Kernel, bool TA, bool TB>
int launch_ws_one(const GemmArgs<double>& a, cudaStream_t stream) {
  static std::atomic<bool> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return B2_ERR_LAUNCH;
  auto kfn = gemm_ws_kernel<Kernel>;
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Kernel::SMEM_BYTES) !=
        cudaSuccess)
      return B2_ERR_LAUNCH;
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  int* status = status_pointer();
  if (!status) return B2_ERR_LAUNCH;
  CUtensorMap mapA, mapB;
  const int64_t ra = TA ? a.k : a.m, ca = TA ? a.m : a.k;  // stored shape of A
  const int64_t rb = TB ? a.n : a.k, cb = TB ? a.k : a.n;  // stored shape of B
  if (!make_map(&mapA, a.A, ra, ca, a.lda, Kernel::A_INNER, Kernel::A_OUTER)) return B2_ERR_LAUNCH;
  if (!make_map(&mapB, a.B, rb, cb, a.ldb, Kernel::B_INNER, Kernel::B_OUTER)) return B2_ERR_LAUNCH;
  const long long tiles = (long long)a.tiles_m * a.tiles_n;
  if (tiles <= 0 || tiles > 0x7fffffffLL) return B2_ERR_LAUNCH;
  // one resident CTA per SM (the rings take most of its shared memory); fewer when there are fewer tiles
  const long long sms = sm_count_cached();
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  kfn<<<grid, Kernel::NT, Kernel::SMEM_BYTES, stream>>>(a, mapA, mapB, status);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

template <template <bool, bool> class MicroT, int GROUPS, int GSTAGES, int CR, int PR, bool STAGE_C>
int launch_ws(const GemmArgs<double>& args_in, bool ta, bool tb, bool aligned, cudaStream_t s) {
  // tensor maps need 16-byte aligned bases and row pitches; coordinates are 32-bit; one problem, all of C, no split
  if (!aligned || args_in.batch > 1 || args_in.ksplit > 1 || args_in.tri != 0) return B2_ERR_VARIANT;
  if (args_in.m > 0x7fffffffLL || args_in.n > 0x7fffffffLL || args_in.k > 0x7fffffffLL) return B2_ERR_VARIANT;
  GemmArgs<double> a = args_in;
  constexpr int BM = MicroT<false, false>::BM, BN = MicroT<false, false>::BN;
  a.tiles_m = (int)((a.m + BM - 1) / BM);
  a.tiles_n = (int)((a.n + BN - 1) / BN);
  if (a.group_m <= 0) a.group_m = 8;
  if (!ta && !tb) return launch_ws_one<GemmWsKernel<MicroT<false, false>, GROUPS, GSTAGES, false, false, CR, PR, STAGE_C>, false, false>(a, s);
  if (!ta && tb) return launch_ws_one<GemmWsKernel<MicroT<false, true>, GROUPS, GSTAGES, false, true, CR, PR, STAGE_C>, false, true>(a, s);
  if (ta && !tb) return launch_ws_one<GemmWsKernel<MicroT<true, false>, GROUPS, GSTAGES, true, false, CR, PR, STAGE_C>, true, false>(a, s);
  return launch_ws_one<GemmWsKernel<MicroT<true, true>, GROUPS, GSTAGES, true, true, CR, PR, STAGE_C>, true, true>(a, s);
}

template <bool TA, bool TB>
using MicroWs64 = DmmaMicro<64, 64, 16, 2, 2, TA, TB>;  // a group: 4 warps of 32 x 32

}  // namespace

// three groups on 64 x 64 tiles with 3-slab rings (3 x 3 x 19 KB), one staging tile for the results (33 KB) and a
// producer warp: 512 threads launched with 128 registers, split 3 x 152 + 40 = 496 <= 4 x 128
int launch_f64_ws_64x64(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_ws<MicroWs64, 3, 3, 152, 40, true>(a, ta, tb, aligned, s);
}
// the same with the micro-kernel's epilogue (stores from registers): the measured counterpart
int launch_f64_ws_64x64_direct(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_ws<MicroWs64, 3, 3, 152, 40, false>(a, ta, tb, aligned, s);
}

}  // namespace b2
