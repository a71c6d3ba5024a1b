// fp32 variant 3: scalar FFMA outer products, 128 x 64 x 16 CTA tile, 4 warps, 4-stage ring, 4 CTAs/SM.
// Kept as the one-multiply-add-per-instruction counterpart the packed-pair variants are measured against.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32V3 = SimtMicro<float, 128, 64, 16, 2, 2, TA, TB, false>;
int launch_f32_v3(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32V3, 4, 4>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
