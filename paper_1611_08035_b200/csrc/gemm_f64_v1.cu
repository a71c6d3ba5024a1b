// fp64 variant 1: DMMA, 128 x 64 x 16 CTA tile, 4 warps of 64 x 32, 3-stage ring, 2 CTAs/SM.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64V1 = DmmaMicro<128, 64, 16, 2, 2, TA, TB>;
int launch_f64_v1(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64V1, 3, 2>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
