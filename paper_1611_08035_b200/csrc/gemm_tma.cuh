// The fp64 tensor-core GEMM kernel with TMA staging: the same tile loop, micro-kernel and
// epilogue as gemm_kernel.cuh, but the operand slabs are brought into shared memory by the
// tensor memory accelerator (cp.async.bulk.tensor) and handed from producer to consumers
// through mbarriers instead of cp.async groups and a CTA-wide barrier per slab.
//
// Why it fits: the DMMA micro-kernel reads either shared-memory layout, and both layouts are
// dense boxes whose inner extent is the tile extent plus a few elements of padding (pitch =
// 4 or 2 mod 16 doubles keeps every fragment load bank-conflict free).  So one TMA box per
// operand per slab, with an inner extent of pitch elements, reproduces the staged tile exactly;
// the few extra elements it fetches belong to the neighbouring tile and are never read.  TMA
// zero-fills whatever lies outside the matrix, which covers edge tiles and the partial last
// k-slab with no extra code (the paper's "packing" step, Section 2.1, done by hardware).
//
// Requirements (checked on the host): A and B 16-byte aligned with even leading dimensions.
// Every wait on an mbarrier is bounded; when a bound is hit the kernel records
// B2_ERR_TIMEOUT in a status word, stops computing, waits (bounded) for the copies it still
// has in flight and returns.
#pragma once
#include <cuda.h>

#include "gemm_kernel.cuh"

namespace b2 {

// ---- mbarrier / TMA primitives -------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done != 0;
}
// Non-blocking test of a phase (try_wait may suspend the thread for a while; a thread that polls several
// barriers in turn must not).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done != 0;
}
// Bounded wait: false when the phase did not complete within limit_ns nanoseconds of wall time.  The bound is a
// time (the global nanosecond timer), not a number of polls, because one try_wait may itself block for an
// implementation-defined interval.  A wait that succeeds at once never reads the timer; after that the timer is
// read once per 32 polls.  kWaitLimitNs is far beyond any legitimate wait of these kernels (a slab arrives within
// microseconds) and still bounds a stuck CTA to about a second; kDrainLimitNs bounds the waits for copies that are
// already in flight when a kernel gives up.
constexpr uint64_t kWaitLimitNs = 1000ull * 1000 * 1000;
constexpr uint64_t kDrainLimitNs = 50ull * 1000 * 1000;
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  do {
#pragma unroll 1
    for (int poll = 0; poll < 32; ++poll)
      if (mbar_try_wait(bar, parity)) return true;
  } while (global_timer_ns() - t0 < limit_ns);
  return false;
}
// One 2-D box from global (through the tensor map) to shared memory, completion counted on `bar`.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int c_inner, int c_outer,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c_inner), "r"(c_outer),
      "r"(smem_u32(bar))
      : "memory");
}

// ---- untiled bulk copies (both addresses 16-byte aligned, size a multiple of 16 bytes) ---------------------
// global -> shared, completion counted on `bar`
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// all of this thread's bulk stores have completed (bulk_wait_read_all: have read their source)
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- host helpers shared by the TMA-staged kernels (defined in gemm_f64_tma.cu) ------------------
// 2-D fp64 tensor map of a column-major matrix (rows contiguous, leading dimension ld) with the given box.
bool make_map(CUtensorMap* map, const double* base, int64_t rows, int64_t cols, int64_t ld, int box_inner,
              int box_outer);
// The same for fp32; swizzle64: the 16-byte pieces of every 64-byte box row are permuted (piece index XOR bits
// 7-8 of the shared-memory address), so that pieces of consecutive rows fall into different banks.
bool make_map_f32(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t ld, int box_inner,
                  int box_outer, bool swizzle64);
// Device address (on the current device) of the status word that bounded waits write; nullptr on failure.
int* status_pointer();

// ---- the kernel ------------------------------------------------------------------------------
// LAG: the producer refills, before it multiplies slab kt, the slot of slab kt - LAG, so STAGES - LAG slabs are in
// flight or ready.  With LAG = 1 the producing thread waits at every slab until the slowest warp of the CTA has
// released the slab just finished, and its own warp with it; LAG = 2 asks for a slot that all warps left a whole
// slab ago.
template <class Micro, int STAGES, bool TA, bool TB, int LAG = 1>
struct GemmTmaKernel {
  static_assert(LAG >= 1 && LAG < STAGES, "at least one slab must be in flight");
  using T = typename Micro::T;
  static constexpr int BM = Micro::BM, BN = Micro::BN, BK = Micro::BK, NT = Micro::NT;
  static constexpr int NWARPS = NT / 32;
  // boxes: inner extent = shared-memory pitch, outer extent = number of lines of the staged tile
  static constexpr int A_INNER = Micro::PA, A_OUTER = TA ? BM : BK;
  static constexpr int B_INNER = Micro::PB, B_OUTER = TB ? BK : BN;
  static_assert(A_INNER * A_OUTER == Micro::A_STAGE && B_INNER * B_OUTER == Micro::B_STAGE, "boxes tile the stages");
  static constexpr uint32_t A_BYTES = Micro::A_STAGE * sizeof(T), B_BYTES = Micro::B_STAGE * sizeof(T);
  // swizzled boxes (fp32, k-contiguous operands) repeat their pattern every 512 bytes: stages start on 1024
  static constexpr uint32_t ALIGN = sizeof(T) == 4 ? 1024 : 128;
  static_assert(A_BYTES % ALIGN == 0 && B_BYTES % ALIGN == 0, "stages must keep their alignment");
  static constexpr size_t SMEM_BYTES =
      (size_t)STAGES * (A_BYTES + B_BYTES) + 2 * STAGES * sizeof(uint64_t) + (ALIGN > 128 ? ALIGN : 0);

  static __device__ __forceinline__ void run(const GemmArgs<T>& p, const CUtensorMap* mapA, const CUtensorMap* mapB,
                                             int* status) {
    extern __shared__ __align__(128) unsigned char smem_dyn[];
    unsigned char* smem_raw = smem_dyn;
    if constexpr (ALIGN > 128) smem_raw += (ALIGN - (smem_u32(smem_dyn) & (ALIGN - 1))) & (ALIGN - 1);
    T* sA = reinterpret_cast<T*>(smem_raw);
    T* sB = sA + STAGES * Micro::A_STAGE;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + (size_t)STAGES * (A_BYTES + B_BYTES));
    uint64_t* empty = full + STAGES;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int warp_m = warp % (BM / Micro::WTM), warp_n = warp / (BM / Micro::WTM);

    int tm, tn;
    tile_coords(blockIdx.x, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
    const int64_t m0 = (int64_t)tm * BM, n0 = (int64_t)tn * BN;
    if (tile_outside_triangle(p.tri, m0, n0, BM, BN)) return;  // triangular update: nothing of this tile is stored
    const int KT = (int)((p.k + BK - 1) / BK);

    if (tid == 0) {
      for (int s = 0; s < STAGES; ++s) {
        mbar_init(&full[s], 1);        // one arrival (the producer's expect_tx) plus the bytes of both boxes
        mbar_init(&empty[s], NWARPS);  // one arrival per consumer warp
      }
      mbar_fence_init();
    }
    __syncthreads();

    // producer (thread 0): slab kt goes to slot kt % STAGES
    auto issue = [&](int kt) {
      const int slot = kt % STAGES;
      const int k0 = kt * BK;
      mbar_arrive_expect_tx(&full[slot], A_BYTES + B_BYTES);
      tma_load_2d(sA + slot * Micro::A_STAGE, mapA, TA ? k0 : (int)m0, TA ? (int)m0 : k0, &full[slot]);
      tma_load_2d(sB + slot * Micro::B_STAGE, mapB, TB ? (int)n0 : k0, TB ? k0 : (int)n0, &full[slot]);
    };

    int issued = 0;  // slabs handed to the TMA so far (thread 0 only)
    if (tid == 0) {
      for (; issued < STAGES - LAG && issued < KT; ++issued) issue(issued);
    }

    // beta == 1 or 0, interior tile, 16-byte aligned columns of C: the tile will leave through shared memory and be
    // ADDED to C in memory, or stored, by bulk copies (drain_by_reduction in gemm_kernel.cuh)
    constexpr bool REDUCE_OK = (size_t)STAGES * (A_BYTES + B_BYTES) >= (size_t)Micro::BN * Micro::PC * sizeof(T);
    const bool by_reduction = REDUCE_OK && tile_added_in_memory<Micro>(p, p.C, m0, n0);

    // beta != 0: pull the tile's old C values towards L2 while the k-loop runs (not for a tile that is added in
    // memory: no thread will wait for those values, and the update measures 2 % faster without the prefetch)
    if (p.beta != T(0) && !by_reduction) {
      const int m_valid = (int)min((int64_t)BM, p.m - m0), n_valid = (int)min((int64_t)BN, p.n - n0);
      constexpr int LINE = 16, LPC = (BM + LINE - 1) / LINE;
      for (int c = tid; c < BN * LPC; c += NT) {
        const int col = c / LPC, row = (c % LPC) * LINE;
        if (col < n_valid && row < m_valid) {
          const T* ptr = p.C + (n0 + col) * p.ldc + m0 + row;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
        }
      }
    }

    typename Micro::Acc acc;
    Micro::zero(acc);

    bool ok = true;
    int waited = 0;  // slabs whose arrival this thread has seen
    for (int kt = 0; kt < KT; ++kt) {
      const int slot = kt % STAGES;
      // refill the slot that slab kt - LAG used, once every warp has released it
      if (tid == 0 && issued < KT) {
        const int fslot = issued % STAGES;
        const int round = issued / STAGES;  // how many times this slot has been filled before
        if (round > 0 && !mbar_wait_bounded(&empty[fslot], (uint32_t)((round - 1) & 1))) {
          ok = false;
        } else {
          issue(issued);
          ++issued;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;  // thread 0's verdict reaches the rest of warp 0
      if (!ok) break;
      if (!mbar_wait_bounded(&full[slot], (uint32_t)((kt / STAGES) & 1))) {
        ok = false;
        break;
      }
      waited = kt + 1;
      Micro::compute(acc, sA + slot * Micro::A_STAGE, sB + slot * Micro::B_STAGE, warp_m, warp_n, lane);
      // The fragment loads above went through the generic proxy; the refill of this slot is written by the
      // async proxy.  Accesses to one location through two proxies are ordered only by a proxy fence, and the
      // mbarrier hand-off alone does not supply it: without this fence the refill was observed (rarely, a
      // few tiles in 65536) to land before a warp's last fragment loads of the slab it replaces.
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[slot]);
    }

    if (!ok) {
      // A bounded wait ran out: record it, let the copies still in flight land (their slots have not been
      // refilled since, so the parity of their phase is unambiguous), and leave without storing anything.
      atomicExch(status, (int)B2_ERR_TIMEOUT);
      if (tid == 0) {
        for (int kt = waited; kt < issued; ++kt)
          (void)mbar_wait_bounded(&full[kt % STAGES], (uint32_t)((kt / STAGES) & 1), kDrainLimitNs);
      }
      return;
    }
    if constexpr (REDUCE_OK) {
      if (by_reduction) {
        drain_by_reduction<Micro>(acc, p, p.C, m0, n0, reinterpret_cast<T*>(smem_raw), warp_m, warp_n, lane);
        return;
      }
    }
    if (tile_crosses_diagonal(p.tri, m0, n0, BM, BN)) {
      Micro::epilogue_masked(acc, p, p.C, m0, n0, warp_m, warp_n, lane);
    } else {
      Micro::epilogue(acc, p, p.C, m0, n0, warp_m, warp_n, lane);
    }
  }
};

template <class Kernel, int MIN_CTAS>
__global__ void __launch_bounds__(Kernel::NT, MIN_CTAS)
    gemm_tma_kernel(const GemmArgs<typename Kernel::T> p, const __grid_constant__ CUtensorMap mapA,
                    const __grid_constant__ CUtensorMap mapB, int* status) {
  Kernel::run(p, &mapA, &mapB, status);
}

}  // namespace b2
