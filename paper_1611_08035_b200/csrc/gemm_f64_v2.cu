// fp64 variant 2: DMMA, 64 x 64 x 16 CTA tile, 4 warps of 32 x 32, 3-stage ring, 4 CTAs/SM
// (small problems: more tiles to fill the SMs).
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64V2 = DmmaMicro<64, 64, 16, 2, 2, TA, TB>;
int launch_f64_v2(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64V2, 3, 4>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
