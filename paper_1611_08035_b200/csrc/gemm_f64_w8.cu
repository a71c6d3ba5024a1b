// fp64 variant with eight warps on a 64 x 64 x 16 tile (cp.async staging): warps of 32 x 16, about 80 registers,
// 3 CTAs/SM.  Twice the warps per tile of the four-warp kernel at the price of one more fragment load per four
// tensor-core instructions: for problems whose 64 x 64 tiles are fewer than the SMs can hold, where the
// four-warp kernel leaves the schedulers with one or two warps each.
#include "gemm_launch.cuh"
namespace b2 {
template <bool TA, bool TB>
using MicroF64W8 = DmmaMicro<64, 64, 16, 2, 4, TA, TB>;
int launch_f64_w8(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return VariantLauncher<MicroF64W8, 3, 3>::launch(a, ta, tb, aligned, s);
}
}  // namespace b2
