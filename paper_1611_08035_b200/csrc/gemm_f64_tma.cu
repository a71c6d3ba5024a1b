// fp64 DMMA kernels with TMA staging (variants 4-6, 8): tensor-map encoding, launch, device status word.
#include <cuda.h>
#include <cuda_runtime.h>

#include "b2gemm.h"
#include "gemm_launch.cuh"
#include "gemm_tma.cuh"

namespace b2 {
int tf32_take_status();  // status word of the TF32 tensor-core kernels (sgemm_tf32.cu)
namespace {

// Status word the TMA kernels write when a bounded wait runs out; read and cleared by b2_device_status.
__device__ int g_device_status = 0;

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn lookup_encode_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return reinterpret_cast<EncodeFn>(p);
  return nullptr;
}
EncodeFn encode_fn() {
  static const EncodeFn fn = lookup_encode_fn();  // initialised once, thread-safe
  return fn;
}

}  // namespace

// 2-D fp64 tensor map of a column-major matrix (rows contiguous) with the given box.
bool make_map(CUtensorMap* map, const double* base, int64_t rows, int64_t cols, int64_t ld, int box_inner,
              int box_outer) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)rows, (cuuint64_t)cols};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(double)};
  const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<double*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map_f32(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t ld, int box_inner,
                  int box_outer, bool swizzle64) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)rows, (cuuint64_t)cols};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int* status_pointer() {
  static std::atomic<int*> by_device[64];  // concurrent first calls store the same address
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  int* cached = by_device[dev].load(std::memory_order_acquire);
  if (!cached) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
    cached = static_cast<int*>(p);
    by_device[dev].store(cached, std::memory_order_release);
  }
  return cached;
}

namespace {

template <class Kernel, int MIN_CTAS, bool TA, bool TB>
int launch_tma_one(const GemmArgs<double>& a, cudaStream_t stream) {
  static std::atomic<bool> configured[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return B2_ERR_LAUNCH;
  auto kfn = gemm_tma_kernel<Kernel, MIN_CTAS>;
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Kernel::SMEM_BYTES) !=
        cudaSuccess)
      return B2_ERR_LAUNCH;
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  int* status = status_pointer();
  if (!status) return B2_ERR_LAUNCH;
  CUtensorMap mapA, mapB;
  const int64_t ra = TA ? a.k : a.m, ca = TA ? a.m : a.k;  // stored shape of A
  const int64_t rb = TB ? a.n : a.k, cb = TB ? a.k : a.n;  // stored shape of B
  if (!make_map(&mapA, a.A, ra, ca, a.lda, Kernel::A_INNER, Kernel::A_OUTER)) return B2_ERR_LAUNCH;
  if (!make_map(&mapB, a.B, rb, cb, a.ldb, Kernel::B_INNER, Kernel::B_OUTER)) return B2_ERR_LAUNCH;
  const long long tiles = (long long)a.tiles_m * a.tiles_n;
  if (tiles <= 0 || tiles > 0x7fffffffLL) return B2_ERR_LAUNCH;
  kfn<<<(unsigned)tiles, Kernel::NT, Kernel::SMEM_BYTES, stream>>>(a, mapA, mapB, status);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

template <template <bool, bool> class MicroT, int STAGES, int MIN_CTAS>
int launch_tma(const GemmArgs<double>& args_in, bool ta, bool tb, bool aligned, cudaStream_t s) {
  // tensor maps need 16-byte aligned bases and row pitches; coordinates are 32-bit
  if (!aligned || args_in.batch > 1 || args_in.ksplit > 1) return B2_ERR_VARIANT;
  if (args_in.m > 0x7fffffffLL || args_in.n > 0x7fffffffLL || args_in.k > 0x7fffffffLL) return B2_ERR_VARIANT;
  GemmArgs<double> a = args_in;
  constexpr int BM = MicroT<false, false>::BM, BN = MicroT<false, false>::BN;
  a.tiles_m = (int)((a.m + BM - 1) / BM);
  a.tiles_n = (int)((a.n + BN - 1) / BN);
  if (a.group_m <= 0) a.group_m = 8;
  if (!ta && !tb) return launch_tma_one<GemmTmaKernel<MicroT<false, false>, STAGES, false, false>, MIN_CTAS, false, false>(a, s);
  if (!ta && tb) return launch_tma_one<GemmTmaKernel<MicroT<false, true>, STAGES, false, true>, MIN_CTAS, false, true>(a, s);
  if (ta && !tb) return launch_tma_one<GemmTmaKernel<MicroT<true, false>, STAGES, true, false>, MIN_CTAS, true, false>(a, s);
  return launch_tma_one<GemmTmaKernel<MicroT<true, true>, STAGES, true, true>, MIN_CTAS, true, true>(a, s);
}

// Waits, with a short bound, on a barrier that nothing ever completes: exercises the time-out path
// (status word, clean return) without faulting or hanging anything.
__global__ void wait_timeout_selftest_kernel(int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncthreads();
  // one millisecond, then give up
  if (threadIdx.x == 0 && !mbar_wait_bounded(&bar, 0, 1000ull * 1000)) atomicExch(status, (int)B2_ERR_TIMEOUT);
}

template <bool TA, bool TB>
using MicroTma64 = DmmaMicro<64, 64, 16, 2, 2, TA, TB>;
template <bool TA, bool TB>
using MicroTma128x64 = DmmaMicro<128, 64, 16, 2, 2, TA, TB>;
template <bool TA, bool TB>
using MicroTma128 = DmmaMicro<128, 128, 16, 2, 4, TA, TB>;
template <bool TA, bool TB>
using MicroTmaT32 = DmmaMicro<32, 32, 16, 2, 2, TA, TB>;  // 4 warps of 16 x 16

}  // namespace

int launch_f64_v4(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_tma<MicroTma64, 3, 4>(a, ta, tb, aligned, s);
}
int launch_f64_v5(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_tma<MicroTma128x64, 3, 2>(a, ta, tb, aligned, s);
}
int launch_f64_v6(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_tma<MicroTma128, 4, 1>(a, ta, tb, aligned, s);
}
int launch_f64_tma_t32(const GemmArgs<double>& a, bool ta, bool tb, bool aligned, cudaStream_t s) {
  return launch_tma<MicroTmaT32, 3, 6>(a, ta, tb, aligned, s);
}

}  // namespace b2

extern "C" int b2_selftest_wait_timeout(void* cuda_stream) {
  int* status = b2::status_pointer();
  if (!status) return B2_ERR_LAUNCH;
  b2::wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

extern "C" int b2_device_status(void* cuda_stream) {
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return B2_ERR_LAUNCH;
  int value = 0;
  if (cudaMemcpyFromSymbol(&value, b2::g_device_status, sizeof(int)) != cudaSuccess) return B2_ERR_LAUNCH;
  if (value != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(b2::g_device_status, &zero, sizeof(int)) != cudaSuccess) return B2_ERR_LAUNCH;
  }
  const int other = b2::tf32_take_status();
  return value != 0 ? value : other;
}
