// fp32 variant 1: packed-pair FMA outer products, 128 x 64 x 16 CTA tile, 4 warps, 8 x 8 accumulators per thread,
// 4-stage ring, 3 CTAs/SM (168 registers: room to double-buffer the fragments).  A k-contiguous B (NN, TN) is
// transposed through registers instead of by 4-byte cp.async (NN 8192^3: 59.2 against 57.9 TFLOP/s).
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32V1 = SimtMicro<float, 128, 64, 16, 2, 2, TA, TB, true, 8, 8, true>;
int launch_f32_v1(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32V1, 4, 3>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
