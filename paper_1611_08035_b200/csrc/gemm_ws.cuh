// The fp64 tensor-core GEMM as a persistent, warp-specialised kernel.
//
// The paper's view of the k-loop (Section 1): ramp-up, steady state, drain -- and only the steady state runs the
// arithmetic pipe at its rate.  With one CTA per tile every tile pays its own ramp-up (the first operand slabs
// have to arrive) and drain (the C tile is read, updated and written) with the pipe idle unless another CTA on
// the same SM happens to be in its steady state; when k is short (a rank-k update with k = 64 is four slabs)
// those two phases are most of a CTA's life.  Here one CTA per SM stays resident and walks over its share of
// the tiles, and the phases are given to different warps so that they overlap by construction:
//
//   - a producer warp (one thread issues) streams the operand slabs of the coming tiles through per-group rings
//     in shared memory with the tensor memory accelerator; it runs ahead across tile boundaries, so a group's
//     next tile is (being) staged while its current tile is multiplied: the ramp-up disappears;
//   - GROUPS groups of four warps each own one 64 x 64 tile at a time, with the DMMA micro-kernel of
//     gemm_kernel.cuh (same fragments, same shared-memory layouts).  The groups work on different tiles and start
//     a fraction of a tile apart, so while one group drains the others keep the tensor pipe busy;
//   - the drain's stores do not go through the load/store unit (global stores issued by the multiplying warps
//     were measured to hold up the fragment loads of the other groups: a tenth of the run time of a k = 64 update):
//     a group writes alpha*acc + beta*C into a staging tile in shared memory, and its first 64 threads send one
//     column each back to C with a bulk copy.  The CTA has one staging tile; the groups use it in the order of the
//     CTA's tile list.  (Tiles on the edge of C and a C without 16-byte aligned columns use the micro-kernel's
//     general epilogue instead.)
//   - Tiles are handed out in rasterised order, CTA b taking tiles b, b + gridDim.x, ... (the tiles of one
//     problem cost the same, so a fixed round-robin is balanced to within one tile per CTA), group g of a CTA
//     every GROUPS-th of those.
//
// Hand-off barriers (mbarriers in shared memory): per group and ring slot "full" (the producer's expect_tx plus
// the bytes of both boxes) and "empty" (one arrival per warp of the group, after a proxy fence: the slot was read
// through the generic proxy and is overwritten through the async proxy); per group "cdone" (every warp has put its
// results into the staging tile) and "sfree" (the bulk stores of the group's tile have read the staging tile out:
// one arrival per column owner).  Every wait is bounded in time; when a bound is hit the
// thread records B2_ERR_TIMEOUT in the status word and stops working, and the producer waits (bounded) for the
// copies it still has in flight before it leaves.
//
// Registers.  A CTA's warps are spread over the SM's four sub-partitions, each with a quarter of the register
// file, so what a thread may have is set by the warps per sub-partition: GROUPS + 1 warpgroups of four warps put
// GROUPS + 1 warps on each.  The kernel is launched with the even share and then moves registers from the
// producer's warpgroup (which needs few) to the multiplying ones with setmaxnreg; CONSUMER_REGS and PRODUCER_REGS
// (multiples of 8) must add up to no more than the launch's total:
//     GROUPS * CONSUMER_REGS + PRODUCER_REGS <= (GROUPS + 1) * launch registers per thread.
//
// Requirements (checked on the host): A and B 16-byte aligned with even leading dimensions, a single problem
// (no batch), the whole of C (no triangle), no k split.
#pragma once
#include "gemm_tma.cuh"

namespace b2 {

template <int REGS>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
}
template <int REGS>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}

template <class Micro, int GROUPS, int GSTAGES, bool TA, bool TB, int CONSUMER_REGS, int PRODUCER_REGS, bool STAGE_C>
struct GemmWsKernel {
  using T = double;
  static_assert(std::is_same<typename Micro::T, double>::value, "instantiated for the fp64 DMMA micro-kernel");
  static constexpr int BM = Micro::BM, BN = Micro::BN, BK = Micro::BK;
  static constexpr int GT = Micro::NT;  // threads of one group
  static constexpr int GW = GT / 32;    // warps of one group
  static_assert(GT == 128 && BM == 64 && BN == 64, "groups of four warps (one warpgroup) on 64 x 64 tiles");
  static constexpr int NT = (GROUPS + 1) * GT;  // plus the producer's warpgroup (one of its threads works)
  // registers per thread at launch: the even share of a sub-partition's 16384, in the allocation unit of 8
  static constexpr int LAUNCH_REGS = (16384 / (32 * (GROUPS + 1))) / 8 * 8;
  static_assert(CONSUMER_REGS % 8 == 0 && PRODUCER_REGS % 8 == 0 && PRODUCER_REGS >= 24 && CONSUMER_REGS <= 232 &&
                    GROUPS * CONSUMER_REGS + PRODUCER_REGS <= (GROUPS + 1) * LAUNCH_REGS,
                "the register split must fit the registers the block is launched with");
  static constexpr int A_INNER = Micro::PA, A_OUTER = TA ? BM : BK;
  static constexpr int B_INNER = Micro::PB, B_OUTER = TB ? BK : BN;
  static_assert(A_INNER * A_OUTER == Micro::A_STAGE && B_INNER * B_OUTER == Micro::B_STAGE, "boxes tile the stages");
  static constexpr uint32_t A_BYTES = Micro::A_STAGE * 8, B_BYTES = Micro::B_STAGE * 8;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static_assert(A_BYTES % 128 == 0 && B_BYTES % 128 == 0, "stages must keep 128-byte alignment");
  // Staging tile for results, column by column with a pitch of 2 (mod 8) doubles: a column starts on a 16-byte
  // boundary (bulk copies), and the fragment stores (a lane's two adjacent rows of one column, eight lanes down a
  // column, four columns two apart) are free of bank conflicts.
  static constexpr int C_PITCH = BM + 2;
  static constexpr uint32_t CBUF_BYTES = STAGE_C ? BN * C_PITCH * 8 : 0;
  static constexpr uint32_t COL_BYTES = BM * 8;
  // old C values of a tile are requested in this many batches (one: all 32 values of a thread in flight at once)
  static constexpr int C_BATCHES = CONSUMER_REGS >= 152 ? 1 : 2;
  static constexpr size_t RING_BYTES = (size_t)GROUPS * GSTAGES * STAGE_BYTES;
  static constexpr int NBARS = 2 * GROUPS * GSTAGES + 3 * GROUPS;  // full, empty; cdone, stagger, sfree
  static constexpr size_t BAR_OFFSET = RING_BYTES + CBUF_BYTES;
  static constexpr size_t SMEM_BYTES = BAR_OFFSET + NBARS * sizeof(uint64_t);

  static __device__ __forceinline__ void run(const GemmArgs<T>& p, const CUtensorMap* mapA, const CUtensorMap* mapB,
                                             int* status) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + BAR_OFFSET);
    uint64_t* empty = full + GROUPS * GSTAGES;
    uint64_t* cdone = empty + GROUPS * GSTAGES;
    uint64_t* stagger = cdone + GROUPS;
    uint64_t* sfree = stagger + GROUPS;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int KT = (int)((p.k + BK - 1) / BK);
    const int tiles_total = p.tiles_m * p.tiles_n;
    // tiles of this CTA: blockIdx.x + i*gridDim.x, i = 0 .. my_tiles-1; group g takes i = g, g + GROUPS, ...
    const int my_tiles = (tiles_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (tid == 0) {
      for (int s = 0; s < GROUPS * GSTAGES; ++s) {
        mbar_init(&full[s], 1);    // the producer's expect_tx arrival plus the bytes of both boxes
        mbar_init(&empty[s], GW);  // one arrival per warp of the group
      }
      for (int s = 0; s < GROUPS; ++s) {
        mbar_init(&cdone[s], GW);    // one arrival per warp: its results are in the staging tile
        mbar_init(&stagger[s], GW);  // arrivals: the warps of group 0
      }
      for (int s = 0; s < GROUPS; ++s) mbar_init(&sfree[s], BN);  // one arrival per column owner of group s
      mbar_fence_init();
    }
    __syncthreads();

    auto tile_origin = [&](int i, int& m0, int& n0) {
      int tm, tn;
      tile_coords((int)blockIdx.x + i * (int)gridDim.x, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
      m0 = tm * BM, n0 = tn * BN;
    };

    if (warp >= GROUPS * GW) {
      // ---------------- producer ----------------
      setmaxnreg_dec<PRODUCER_REGS>();  // the whole warpgroup gives its surplus to the multiplying groups
      if (tid != GROUPS * GT) return;
      int tile_i[GROUPS], kt[GROUPS], cnt[GROUPS];  // next tile (index into the CTA's list), next slab, slabs issued
      int m0[GROUPS], n0[GROUPS];
#pragma unroll
      for (int g = 0; g < GROUPS; ++g) {
        tile_i[g] = g, kt[g] = 0, cnt[g] = 0, m0[g] = 0, n0[g] = 0;
        if (tile_i[g] < my_tiles) tile_origin(tile_i[g], m0[g], n0[g]);
      }
      bool ok = true;
      uint64_t idle_since = 0;
      for (;;) {
        bool remaining = false, progress = false;
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) {
          if (tile_i[g] >= my_tiles) continue;
          remaining = true;
          const int slot = cnt[g] % GSTAGES, round = cnt[g] / GSTAGES;
          uint64_t* fb = &full[g * GSTAGES + slot];
          if (round > 0 && !mbar_test_wait(&empty[g * GSTAGES + slot], (uint32_t)((round - 1) & 1))) continue;
          unsigned char* dst = smem_raw + (size_t)(g * GSTAGES + slot) * STAGE_BYTES;
          const int k0 = kt[g] * BK;
          mbar_arrive_expect_tx(fb, STAGE_BYTES);
          tma_load_2d(dst, mapA, TA ? k0 : m0[g], TA ? m0[g] : k0, fb);
          tma_load_2d(dst + A_BYTES, mapB, TB ? n0[g] : k0, TB ? k0 : n0[g], fb);
          ++cnt[g];
          progress = true;
          if (++kt[g] == KT) {
            kt[g] = 0;
            tile_i[g] += GROUPS;
            if (tile_i[g] < my_tiles) tile_origin(tile_i[g], m0[g], n0[g]);
          }
        }
        if (!remaining) break;
        if (progress) {
          idle_since = 0;
        } else {
          // every ring is full: the groups are multiplying.  Bound the time without any progress.
          const uint64_t now = global_timer_ns();
          if (idle_since == 0) {
            idle_since = now;
          } else if (now - idle_since > kWaitLimitNs) {
            ok = false;
            break;
          }
          __nanosleep(32);
        }
      }
      if (!ok) {
        atomicExch(status, (int)B2_ERR_TIMEOUT);
        // let the copies still in flight land: the latest fill of every slot
#pragma unroll
        for (int g = 0; g < GROUPS; ++g)
          for (int s = 0; s < GSTAGES; ++s) {
            if (cnt[g] <= s) continue;
            const int last = ((cnt[g] - 1 - s) / GSTAGES) * GSTAGES + s;  // last slab that went to slot s
            (void)mbar_wait_bounded(&full[g * GSTAGES + s], (uint32_t)((last / GSTAGES) & 1), kDrainLimitNs);
          }
      }
      return;
    }

    // ---------------- group g, warps wl = 0 .. GW-1 ----------------
    setmaxnreg_inc<CONSUMER_REGS>();
    const int g = warp / GW, wl = warp % GW;
    constexpr int WM = BM / Micro::WTM;
    const int warp_m = wl % WM, warp_n = wl / WM;
    if (g >= my_tiles) return;  // fewer tiles than groups: nothing for this group
    unsigned char* ring = smem_raw + (size_t)g * GSTAGES * STAGE_BYTES;
    uint64_t* gfull = full + g * GSTAGES;
    uint64_t* gempty = empty + g * GSTAGES;

    // Start the groups a fraction of a tile apart, so that their drains do not coincide from the start: group
    // g > 0 waits until group 0 has finished g/GROUPS of the slabs of its first tile (slab number
    // announce_after(g); -1: at once).
    auto announce_after = [KT](int gg) { return (gg * KT) / GROUPS - 1; };
    bool ok = true;
    if (g > 0) ok = mbar_wait_bounded(&stagger[g], 0);
    if (g == 0 && lane == 0) {
#pragma unroll
      for (int gg = 1; gg < GROUPS; ++gg)
        if (announce_after(gg) < 0) mbar_arrive(&stagger[gg]);
    }

    const bool use_beta = (p.beta != T(0));
    const bool c_vec_ok = ((reinterpret_cast<uintptr_t>(p.C) & 15) == 0) && ((p.ldc & 1) == 0);
    const int gq = lane >> 2, t4 = lane & 3;
    T* cbuf = reinterpret_cast<T*>(smem_raw + RING_BYTES);
    // this thread's first fragment element inside a tile (staging tile and C), and the column it sends back to C
    const int frow = warp_m * Micro::WTM + 2 * gq, fcol = warp_n * Micro::WTN + 2 * t4;
    T* sfrag = cbuf + fcol * C_PITCH + frow;
    const int ltid = wl * 32 + lane;
    const bool owner = ltid < BN;  // (whole warps: the group's first two)

    int cnt = 0;  // slabs consumed by this warp so far
    for (int i = g, u = 0; i < my_tiles && ok; i += GROUPS, ++u) {
      int m0, n0;
      tile_origin(i, m0, n0);
      // beta != 0: pull the tile's old C values towards L2 while the k-loop runs (not when the tile will be added
      // to C in memory: nothing waits for those values then)
      const bool will_add = STAGE_C && c_vec_ok && p.beta == T(1) && (int64_t)m0 + BM <= p.m && (int64_t)n0 + BN <= p.n;
      if (use_beta && !will_add) {
        const int m_valid = (int)min((int64_t)BM, p.m - m0), n_valid = (int)min((int64_t)BN, p.n - n0);
        constexpr int LINE = 16, LPC = BM / LINE;  // 128-byte lines per tile column
        for (int c = ltid; c < BN * LPC; c += GT) {
          const int col = c / LPC, row = (c % LPC) * LINE;
          if (col < n_valid && row < m_valid)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.C + (int64_t)(n0 + col) * p.ldc + m0 + row));
        }
      }
      typename Micro::Acc acc;
      Micro::zero(acc);
      for (int kt = 0; kt < KT; ++kt, ++cnt) {
        const int slot = cnt % GSTAGES;
        if (!mbar_wait_bounded(&gfull[slot], (uint32_t)((cnt / GSTAGES) & 1))) {
          ok = false;
          break;
        }
        const T* sA = reinterpret_cast<const T*>(ring + (size_t)slot * STAGE_BYTES);
        const T* sB = sA + Micro::A_STAGE;
        Micro::compute(acc, sA, sB, warp_m, warp_n, lane);
        // generic-proxy reads of the slot are ordered before its refill through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&gempty[slot]);
          if (g == 0 && i == 0) {
#pragma unroll
            for (int gg = 1; gg < GROUPS; ++gg)
              if (kt == announce_after(gg)) mbar_arrive(&stagger[gg]);
          }
        }
      }
      if (!ok) break;

      // ---- drain: fused alpha/beta epilogue ----
      // through the staging tile when the whole tile lies inside C and its columns are 16-byte aligned
      const bool staged = STAGE_C && c_vec_ok && (int64_t)m0 + BM <= p.m && (int64_t)n0 + BN <= p.n;
      // beta == 1 on a staged tile: nothing of C is loaded; the tile is added to C in memory by bulk reductions
      const bool add_in_memory = staged && p.beta == T(1);
      if (staged) {
        const bool use_beta = p.beta != T(0) && !add_in_memory;
        T* cfrag = p.C + (int64_t)(n0 + fcol) * p.ldc + m0 + frow;
        // results into the accumulator registers; the old values are fetched in C_BATCHES batches
#pragma unroll
        for (int half = 0; half < C_BATCHES; ++half) {
          constexpr int NH = Micro::NI / C_BATCHES;
          double2 old[Micro::MI][NH][2];
          if (use_beta) {
#pragma unroll
            for (int mi = 0; mi < Micro::MI; ++mi)
#pragma unroll
              for (int nj = 0; nj < NH; ++nj)
#pragma unroll
                for (int h = 0; h < 2; ++h)
                  old[mi][nj][h] = *reinterpret_cast<const double2*>(
                      cfrag + (int64_t)((half * NH + nj) * 8 + h) * p.ldc + mi * 16);
          }
#pragma unroll
          for (int mi = 0; mi < Micro::MI; ++mi)
#pragma unroll
            for (int nj = 0; nj < NH; ++nj)
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const int ni = half * NH + nj;
                double v0 = p.alpha * acc.c[mi][ni][h], v1 = p.alpha * acc.c[mi][ni][2 + h];
                if (use_beta) v0 += p.beta * old[mi][nj][h].x, v1 += p.beta * old[mi][nj][h].y;
                acc.c[mi][ni][h] = v0, acc.c[mi][ni][2 + h] = v1;
              }
        }
      } else {
        Micro::epilogue(acc, p, p.C, (int64_t)m0, (int64_t)n0, warp_m, warp_n, lane);
      }
      if constexpr (STAGE_C) {
        // The staging tile is used in the order of the CTA's tile list: tile i may write it once the stores of
        // tile i-1 have read it out (tiles that do not use it pass their turn on).  Tile i-1 belongs to the
        // group before this one; each group announces on a barrier of its own, so a waiting group is never more
        // than one phase away from the phase it asks for (it waited for that group's previous tile one turn ago).
        if (i > 0 && !mbar_wait_bounded(&sfree[(g + GROUPS - 1) % GROUPS], (uint32_t)(((i - 1) / GROUPS) & 1))) {
          ok = false;
          break;
        }
        if (staged) {
#pragma unroll
          for (int mi = 0; mi < Micro::MI; ++mi)
#pragma unroll
            for (int ni = 0; ni < Micro::NI; ++ni)
#pragma unroll
              for (int h = 0; h < 2; ++h)
                *reinterpret_cast<double2*>(sfrag + (ni * 8 + h) * C_PITCH + mi * 16) =
                    make_double2(acc.c[mi][ni][h], acc.c[mi][ni][2 + h]);
          // the results were written through the generic proxy and leave through the async proxy
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&cdone[g]);
        }
        if (owner) {
          if (staged) {
            if (!mbar_wait_bounded(&cdone[g], (uint32_t)(u & 1))) {
              ok = false;
              break;
            }
            if (add_in_memory)
              bulk_reduce_add(p.C + (int64_t)(n0 + ltid) * p.ldc + m0, cbuf + ltid * C_PITCH, COL_BYTES);
            else
              bulk_store(p.C + (int64_t)(n0 + ltid) * p.ldc + m0, cbuf + ltid * C_PITCH, COL_BYTES);
            bulk_commit();
            bulk_wait_read_all();  // the column has left the staging tile
          }
          mbar_arrive(&sfree[g]);
        }
      }
    }
    if (STAGE_C && owner) bulk_wait_all();  // this thread's stores are complete before the CTA's shared memory goes away
    if (!ok && lane == 0) atomicExch(status, (int)B2_ERR_TIMEOUT);
  }
};

template <class Kernel>
__global__ void __launch_bounds__(Kernel::NT, 1)
    gemm_ws_kernel(const GemmArgs<double> p, const __grid_constant__ CUtensorMap mapA,
                   const __grid_constant__ CUtensorMap mapB, int* status) {
  Kernel::run(p, &mapA, &mapB, status);
}

}  // namespace b2
