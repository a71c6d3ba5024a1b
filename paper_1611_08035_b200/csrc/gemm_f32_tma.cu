// fp32 packed-pair kernels with TMA staging: one 128 x 128 tile shape, a micro-kernel per operand layout.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "b2gemm.h"
#include "gemm_f32_tma.cuh"
#include "gemm_launch.cuh"

namespace b2 {
namespace {

template <class Micro, int STAGES, int MIN_CTAS, bool TA, bool TB>
int launch_f32_tma_one(const GemmArgs<float>& a, cudaStream_t stream) {
  using Kernel = GemmTmaKernel<Micro, STAGES, TA, TB, 2>;
  static_assert(Micro::BM == 128 && Micro::BN == 128, "the variant is announced as a 128 x 128 tile");
  static std::atomic<bool> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return B2_ERR_LAUNCH;
  auto kfn = gemm_tma_kernel<Kernel, MIN_CTAS>;
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
  if (!make_map_f32(&mapA, a.A, ra, ca, a.lda, Kernel::A_INNER, Kernel::A_OUTER, Micro::SWIZZLE_A)) return B2_ERR_LAUNCH;
  if (!make_map_f32(&mapB, a.B, rb, cb, a.ldb, Kernel::B_INNER, Kernel::B_OUTER, Micro::SWIZZLE_B)) return B2_ERR_LAUNCH;
  const long long tiles = (long long)a.tiles_m * a.tiles_n;
  if (tiles <= 0 || tiles > 0x7fffffffLL) return B2_ERR_LAUNCH;
  kfn<<<(unsigned)tiles, Kernel::NT, Kernel::SMEM_BYTES, stream>>>(a, mapA, mapB, status);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

}  // namespace

// Per thread: 16 x 8 when A has m contiguous (pairs of rows), 8 x 16 when only B has its C index contiguous (pairs
// of columns).  With both operands k-contiguous (A transposed, B not) no pairing fits: declined.
int launch_f32_tma(const GemmArgs<float>& args_in, bool ta, bool tb, bool aligned, cudaStream_t s) {
  // tensor maps need 16-byte aligned bases and row pitches; coordinates are 32-bit
  // single plain problems only (no batch, no triangle, no k split)
  if (!aligned || args_in.batch > 1 || args_in.ksplit > 1 || args_in.tri != 0 || (ta && !tb)) return B2_ERR_VARIANT;
  if (args_in.m > 0x7fffffffLL || args_in.n > 0x7fffffffLL || args_in.k > 0x7fffffffLL) return B2_ERR_VARIANT;
  GemmArgs<float> a = args_in;
  a.tiles_m = (int)((a.m + 127) / 128);
  a.tiles_n = (int)((a.n + 127) / 128);
  if (a.group_m <= 0) a.group_m = 8;
  if (!ta && tb) return launch_f32_tma_one<SimtTmaMicro<16, 8, 1, 4, false, true>, 6, 2, false, true>(a, s);
  if (!ta && !tb) return launch_f32_tma_one<SimtTmaMicro<16, 8, 1, 4, false, false>, 6, 2, false, false>(a, s);
  return launch_f32_tma_one<SimtTmaMicro<8, 16, 2, 2, true, true>, 6, 2, true, true>(a, s);
}

}  // namespace b2
