// fp32 variant 2: FFMA outer products, 64 x 64 x 16 CTA tile, 2 warps, 4-stage ring, 6 CTAs/SM
// (small problems).
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32V2 = SimtMicro<float, 64, 64, 16, 1, 2, TA, TB>;
int launch_f32_v2(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32V2, 4, 6>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
