// fp32 variant 0: FFMA outer products, 128 x 128 x 16 CTA tile, 8 warps, 8 x 8 per thread,
// 4-stage ring, 2 CTAs/SM.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32V0 = SimtMicro<float, 128, 128, 16, 2, 4, TA, TB>;
int launch_f32_v0(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32V0, 4, 2>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
