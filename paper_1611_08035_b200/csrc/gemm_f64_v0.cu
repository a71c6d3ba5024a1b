// fp64 variant 0: DMMA, 128 x 128 x 16 CTA tile, 8 warps of 64 x 32, 4-stage ring, 1 CTA/SM.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64V0 = DmmaMicro<128, 128, 16, 2, 4, TA, TB>;
int launch_f64_v0(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64V0, 4, 1>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
