// fp32 variant 4, for small problems: 4 x 4 accumulators per thread instead of 8 x 8, 32 x 32 x 16 CTA tile,
// 2 warps, 4-stage ring, 8 CTAs/SM.  A problem that yields only a few 64 x 64 tiles per SM leaves the FP32 pipe
// waiting on shared-memory latency; the small tile gives four times the CTAs and warps (512^3: 20 TFLOP/s
// against 9), at the price of twice the shared-memory traffic per multiply-add.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32S32 = SimtMicro<float, 32, 32, 16, 1, 2, TA, TB, true, 4, 4>;
int launch_f32_s32(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32S32, 4, 8>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
