// fp64 variant 3: scalar DFMA outer products, 128 x 64 x 16 CTA tile, 4 warps, 8 x 8 per thread,
// 3-stage ring, 2 CTAs/SM.  Kept as the FP64-FMA counterpart the tensor-core path is measured against.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64V3 = SimtMicro<double, 128, 64, 16, 2, 2, TA, TB>;
int launch_f64_v3(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64V3, 3, 2>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
