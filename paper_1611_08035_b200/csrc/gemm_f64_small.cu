// fp64 variant for small problems (cp.async staging): a 32 x 32 CTA tile with 4 warps of 16 x 16.  Smaller
// tiles put more CTAs and warps on the SMs when a problem has too few 64 x 64 tiles to fill them.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64T32 = DmmaMicro<32, 32, 16, 2, 2, TA, TB>;
int launch_f64_t32(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64T32, 3, 7>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
