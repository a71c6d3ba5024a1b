// fp32 variant 0: packed-pair FMA outer products, 128 x 128 x 16 CTA tile, 4 warps, 16 x 8 accumulators per
// thread (a warp covers 128 x 32), 3-stage ring, 2 CTAs/SM (about 210 registers per thread).  Per k a lane
// fetches 24 operand values for 128 multiply-adds (8 x 8: 16 for 64), so the shared-memory wavefronts per
// multiply-add drop by a quarter, and an element-wise transposing copy of A or B is spread over twice the tile.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF32V0 = SimtMicro<float, 128, 128, 16, 1, 4, TA, TB, true, 16, 8>;
int launch_f32_v0(const GemmArgs<float>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF32V0, 3, 2>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
