// The GEMM kernel: blocked loop nest, shared-memory staging ("packing"), micro-kernel,
// fringe handling and the fused alpha/beta epilogue.
//
// Structure, following the paper:
//   - Section 2 / Figure 1 (GotoBLAS loop nest as refactored in BLIS): the loops over column
//     panels and row panels of C become the grid of CTA tiles (BM x BN); the kc loop becomes
//     the CTA's loop over BK-deep slabs; packing into per-cache-level buffers becomes a
//     multi-stage cp.async ring in shared memory.
//   - Section 2.1: inside a tile, C(mr x nr) += sum_p a_p b_p^T on register-resident
//     accumulators.  Section 5 (kernel skeleton): zero the accumulators, run the unrolled
//     k-loop of outer products, then add the accumulators into C.
//   - Section 4 ("Dealing with dependencies across pipelines"): the accumulator tile is
//     sized so that every multiply-add of one outer product is independent.
// What the paper leaves out (alpha, beta, transposes, leading dimensions, edge tiles) follows
// the BLAS definition of GEMM.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace b2 {

// Shared-memory layout of a staged operand tile (BO "outer" rows/columns of C by BK of k).
//   OC: [k][o], o contiguous (pitch in elements) -- the paper's packed micro-panel layout
//       (A column-major mr x kc, B row-major kc x nr).
//   KC: [o][k], k contiguous -- the source layout of a transposed A or a non-transposed B,
//       which the tensor-core fragment loads can read directly.
enum Layout { OC = 0, KC = 1 };

// ---------------------------------------------------------------------------------------
// Staging of one BO x BK operand tile from global memory into shared memory with cp.async.
//
// Two paths.  The fast path serves slabs that lie completely inside the operand (the steady
// state of interior tiles): every thread keeps one running source pointer, the chunk
// addresses differ from it by compile-time multiples of one hoisted stride, and nothing is
// predicated.  The general path serves edge tiles and the last, partial k-slab: every chunk
// is clipped against the valid extents, zero-filled beyond them and never read from global.
// VEC is the number of elements per cp.async when source and destination layouts agree
// (16-byte chunks need 16-byte aligned columns); when they differ (k-contiguous source packed
// into the OC layout) the copy is element-wise and transposes on the fly.
// ---------------------------------------------------------------------------------------
template <typename T, int BO, int BK, int NT, Layout SRC, Layout DST, int VEC, int PITCH>
struct Stager {
  static constexpr int ELEM = sizeof(T);
  static constexpr bool STRAIGHT = (SRC == DST);
  static_assert(STRAIGHT || (SRC == KC && DST == OC), "only k-contiguous sources are transposed while staging");
  static constexpr int RUN = 8;  // transposing copy: run length along k handled by consecutive threads
  // straight copy geometry
  static constexpr int CE = (SRC == OC) ? BO : BK;  // contiguous extent
  static constexpr int OE = (SRC == OC) ? BK : BO;  // number of lines
  static constexpr int CPL = CE / VEC;              // chunks per line
  static constexpr int TOTAL = STRAIGHT ? OE * CPL : BO * BK;
  static constexpr int ITER = (TOTAL + NT - 1) / NT;
  static_assert(!STRAIGHT || CE % VEC == 0, "tile extent must be a multiple of the chunk");
  static_assert(TOTAL % NT == 0, "every thread copies the same number of chunks");
  static_assert(!STRAIGHT || NT % CPL == 0, "a line must be covered by consecutive threads of one pass");
  static constexpr int LSTEP = STRAIGHT ? NT / CPL : NT / RUN;  // lines (straight) or o-rows (transposing) per pass
  static constexpr int Q = STRAIGHT ? 1 : BO / LSTEP;           // transposing: passes that cover the o-extent once
  static_assert(STRAIGHT || (NT % RUN == 0 && BO % LSTEP == 0 && BK % RUN == 0), "transposing copy geometry");

  const T* src;  // this thread's first chunk of the next slab to stage (the only per-thread state)

  // element offset of the thread's first chunk inside a stage
  static __device__ __forceinline__ int dst0_of(int tid) {
    if constexpr (STRAIGHT) {
      return (tid / CPL) * PITCH + (tid % CPL) * VEC;
    } else {
      return (tid % RUN) * PITCH + tid / RUN;
    }
  }

  __device__ __forceinline__ void init(const T* X0, int64_t ld, int tid) {
    if constexpr (STRAIGHT) {
      src = X0 + (tid % CPL) * VEC + (int64_t)(tid / CPL) * ld;
    } else {
      src = X0 + (tid % RUN) + (int64_t)(tid / RUN) * ld;
    }
  }

  // advance by one slab (BK along k)
  __device__ __forceinline__ void advance(int64_t ld) { src += (STRAIGHT && SRC == OC) ? (int64_t)BK * ld : (int64_t)BK; }

  // Slab fully inside the operand: no predicates.
  __device__ __forceinline__ void load_fast(T* __restrict__ s, int64_t ld, int tid) const {
    const int64_t lstep = (int64_t)LSTEP * ld;  // source elements between the lines of consecutive passes
    const int dst0 = dst0_of(tid);
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
      if constexpr (STRAIGHT) {
        cp_async_zfill<VEC * ELEM>(s + dst0 + it * LSTEP * PITCH, src + it * lstep, VEC * ELEM);
      } else {
        const int a = it % Q, b = it / Q;
        cp_async_zfill<ELEM>(s + dst0 + b * RUN * PITCH + a * LSTEP, src + a * lstep + b * RUN, ELEM);
      }
    }
  }

  // Edge tile, full slab: only o_valid (< BO) rows/columns of the tile exist.  Chunks that lie entirely outside
  // are skipped, not zero-filled: whatever the shared-memory rows beyond o_valid hold only feeds accumulators of
  // rows/columns >= m or n of C, which the epilogue never stores.  A chunk that straddles the edge copies its
  // valid bytes only.  No address outside the operand is formed into a load.
  __device__ __forceinline__ void load_edge(T* __restrict__ s, int64_t ld, int o_valid, int tid) const {
    const int64_t lstep = (int64_t)LSTEP * ld;
    const int dst0 = dst0_of(tid);
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
      if constexpr (STRAIGHT) {
        if constexpr (SRC == OC) {  // chunk runs along o; every line (k) is valid
          const int nvalid = o_valid - (tid % CPL) * VEC;
          if (nvalid > 0)
            cp_async_zfill<VEC * ELEM>(s + dst0 + it * LSTEP * PITCH, src + it * lstep,
                                       (nvalid < VEC ? nvalid : VEC) * ELEM);
        } else {  // lines are o-rows; chunk runs along k (all valid)
          if (tid / CPL + it * LSTEP < o_valid)
            cp_async_zfill<VEC * ELEM>(s + dst0 + it * LSTEP * PITCH, src + it * lstep, VEC * ELEM);
        }
      } else {
        const int a = it % Q, b = it / Q;
        if (tid / RUN + a * LSTEP < o_valid)
          cp_async_zfill<ELEM>(s + dst0 + b * RUN * PITCH + a * LSTEP, src + a * lstep + b * RUN, ELEM);
      }
    }
  }

  // General path (partial k-slab).  X0 points at element (o0, k0) of the operand; o_valid / k_valid are the
  // numbers of valid rows and k-entries from there; everything beyond is zero-filled.
  static __device__ __noinline__ void load_general(T* __restrict__ s, const T* __restrict__ X0, int64_t ld,
                                                   int o_valid, int k_valid, int tid) {
    if constexpr (STRAIGHT) {
      const int c_valid = (SRC == OC) ? o_valid : k_valid;
      const int l_valid = (SRC == OC) ? k_valid : o_valid;
#pragma unroll 1
      for (int it = 0; it < ITER; ++it) {
        const int c = tid + it * NT;
        const int line = c / CPL;
        const int cc = (c % CPL) * VEC;
        int nvalid = c_valid - cc;
        nvalid = nvalid < 0 ? 0 : (nvalid > VEC ? VEC : nvalid);
        if (line >= l_valid) nvalid = 0;
        const T* g = nvalid > 0 ? X0 + cc + (int64_t)line * ld : X0;
        cp_async_zfill<VEC * ELEM>(s + line * PITCH + cc, g, nvalid * ELEM);
      }
    } else {
#pragma unroll 1
      for (int it = 0; it < ITER; ++it) {
        const int c = tid + it * NT;
        const int kk = (c % RUN) + RUN * (c / (RUN * BO));
        const int o = (c / RUN) % BO;
        const bool ok = (o < o_valid) && (kk < k_valid);
        const T* g = ok ? X0 + kk + (int64_t)o * ld : X0;
        cp_async_zfill<ELEM>(s + kk * PITCH + o, g, ok ? ELEM : 0);
      }
    }
  }
};

// ---------------------------------------------------------------------------------------
// Micro-kernel 1: FP64 tensor-core (DMMA) outer products, mma.sync m16n8k4.
//
// One warp owns a WTM x WTN block of the CTA tile as MI x NI fragments of 16 x 8; each
// mma adds four rank-1 updates (k = 4) to a fragment.  All MI*NI mma of a k-step are
// independent, as the paper's sizing rule asks.
//
// Fragment ownership (lane = 4*g + t, g = 0..7, t = 0..3), PTX m16n8k4 .f64:
//   A (16x4): a0 = (row g, k t), a1 = (row g+8, k t);  B (4x8): b0 = (k t, col g);
//   C (16x8): c0,c1 = (row g, cols 2t, 2t+1), c2,c3 = (row g+8, cols 2t, 2t+1).
// The 16 fragment rows are mapped onto rows of C as  row r -> 2r (r < 8), 2(r-8)+1 (r >= 8),
// so a lane's (a0, a1) are two adjacent rows (one 16-byte shared-memory load in the OC
// layout) and (c0, c2) / (c1, c3) are adjacent rows of one column of C (one 16-byte store).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void dmma_m16n8k4(double (&c)[4], double a0, double a1, double b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k4.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
      : "+d"(c[0]), "+d"(c[1]), "+d"(c[2]), "+d"(c[3])
      : "d"(a0), "d"(a1), "d"(b0));
}

template <int BM_, int BN_, int BK_, int WARPS_M, int WARPS_N, bool TA, bool TB>
struct DmmaMicro {
  using T = double;
  static constexpr int BM = BM_, BN = BN_, BK = BK_;
  static constexpr int NT = 32 * WARPS_M * WARPS_N;
  static constexpr int WTM = BM / WARPS_M, WTN = BN / WARPS_N;
  static constexpr int MI = WTM / 16, NI = WTN / 8;
  static constexpr bool REG_TRANSPOSE_B = false;
  // k split over a cluster: a lane's accumulators as MI*NI*4 64-bit words
  static constexpr bool HAS_KSPLIT = true;
  static constexpr int ACC_WORDS = MI * NI * 4;
  static_assert(WTM % 16 == 0 && WTN % 8 == 0 && BK % 16 == 0, "warp tile must be built from 16x8 fragments");
  // Fragment loads read either layout, so tiles are staged in their source layout.
  static constexpr Layout LA = TA ? KC : OC;
  static constexpr Layout LB = TB ? OC : KC;
  // Pitches (in doubles) that make every fragment load bank-conflict free:
  //   OC: pitch = 4 (mod 16);  KC for A (rows 2g, 2g+1): pitch = 2 (mod 16);  KC for B: 4 (mod 16).
  static constexpr int PA = (LA == OC) ? BM + 4 : BK + 2;
  static constexpr int PB = (LB == OC) ? BN + 4 : BK + 4;
  static constexpr int A_STAGE = (LA == OC) ? BK * PA : BM * PA;
  static constexpr int B_STAGE = (LB == OC) ? BK * PB : BN * PB;
  static constexpr int VEC = 2;

  struct Acc {
    double c[MI][NI][4];
  };

  static __device__ __forceinline__ void zero(Acc& acc) {
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
      for (int ni = 0; ni < NI; ++ni)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc.c[mi][ni][r] = 0.0;
  }
  // word w of the accumulators as bits, and acc[w] += the double held in `bits` (one IEEE addition)
  static __device__ __forceinline__ unsigned long long get_word(const Acc& acc, int w) {
    return (unsigned long long)__double_as_longlong(acc.c[w / (NI * 4)][(w / 4) % NI][w % 4]);
  }
  static __device__ __forceinline__ void add_word(Acc& acc, int w, unsigned long long bits) {
    double& c = acc.c[w / (NI * 4)][(w / 4) % NI][w % 4];
    c = __dadd_rn(c, __longlong_as_double((long long)bits));
  }

  // alpha * acc into a column-major tile in shared memory (column pitch PC, 16-byte aligned columns)
  static constexpr int PC = BM + 2;
  static __device__ __forceinline__ void stage_tile(const Acc& acc, double alpha, double* sC, int warp_m, int warp_n,
                                                    int lane) {
    const int g = lane >> 2, t = lane & 3;
    const int r0 = warp_m * WTM + 2 * g, c0 = warp_n * WTN + 2 * t;
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
      for (int ni = 0; ni < NI; ++ni)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          *reinterpret_cast<double2*>(sC + (c0 + ni * 8 + h) * PC + r0 + mi * 16) =
              make_double2(alpha * acc.c[mi][ni][h], alpha * acc.c[mi][ni][2 + h]);
  }

  // sum of a lane's accumulators (probes keep their result alive through it)
  static __device__ __forceinline__ double checksum(const Acc& acc) {
    double s = 0.0;
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
      for (int ni = 0; ni < NI; ++ni)
#pragma unroll
        for (int r = 0; r < 4; ++r) s += acc.c[mi][ni][r];
    return s;
  }

  // One BK-deep slab: BK/4 k-steps of MI*NI independent mma.
  static __device__ __forceinline__ void compute(Acc& acc, const double* __restrict__ sA,
                                                 const double* __restrict__ sB, int warp_m, int warp_n, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const int wm0 = warp_m * WTM, wn0 = warp_n * WTN;
#pragma unroll
    for (int ks = 0; ks < BK / 4; ++ks) {
      const int kk = ks * 4 + t;
      double a[MI][2], b[NI];
#pragma unroll
      for (int mi = 0; mi < MI; ++mi) {
        const int r = wm0 + mi * 16 + 2 * g;
        if constexpr (LA == OC) {
          const double2 v = *reinterpret_cast<const double2*>(sA + kk * PA + r);
          a[mi][0] = v.x;
          a[mi][1] = v.y;
        } else {
          a[mi][0] = sA[r * PA + kk];
          a[mi][1] = sA[(r + 1) * PA + kk];
        }
      }
#pragma unroll
      for (int ni = 0; ni < NI; ++ni) {
        const int cidx = wn0 + ni * 8 + g;
        b[ni] = (LB == OC) ? sB[kk * PB + cidx] : sB[cidx * PB + kk];
      }
#pragma unroll
      for (int mi = 0; mi < MI; ++mi)
#pragma unroll
        for (int ni = 0; ni < NI; ++ni) dmma_m16n8k4(acc.c[mi][ni], a[mi][0], a[mi][1], b[ni]);
    }
  }

  // C := alpha*acc + beta*C on the warp's block; rows >= m and columns >= n are skipped.
  // The old C values are fetched in batches, all loads of a batch issued before the first
  // store, so their latencies overlap instead of adding up (a store to C may alias a later
  // load of C as far as the compiler can tell).
  static __device__ __forceinline__ void epilogue(const Acc& acc, const GemmArgs<double>& p, double* C, int64_t m0,
                                                  int64_t n0, int warp_m, int warp_n, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((p.ldc & 1) == 0);
    const bool use_beta = (p.beta != 0.0);
    // old values in flight per batch: 32 doubles when the register budget is 255, 16 when it is 128
    constexpr int BATCH = (MI * NI * 4 >= 64) ? 32 : 16;
    constexpr int NB = (BATCH / (MI * 4)) > 0 ? ((BATCH / (MI * 4)) < NI ? (BATCH / (MI * 4)) : NI) : 1;
    static_assert(NI % NB == 0, "batches must tile the fragment columns");
    // this lane's first element, and how many rows / columns of C remain from there (32-bit from here on)
    const int64_t row0 = m0 + warp_m * WTM + 2 * g;
    const int64_t col0 = n0 + warp_n * WTN + 2 * t;
    double* base = C + col0 * p.ldc + row0;
    const int rows_left = (int)min((int64_t)BM, p.m - row0), cols_left = (int)min((int64_t)BN, p.n - col0);
#pragma unroll
    for (int nb0 = 0; nb0 < NI; nb0 += NB) {
      double2 old[NB][2][MI];
      if (use_beta) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int mi = 0; mi < MI; ++mi) {
              const int col = (nb0 + nb) * 8 + h, row = mi * 16;
              old[nb][h][mi] = make_double2(0.0, 0.0);
              if (col < cols_left && row < rows_left) {
                const double* src = base + col * p.ldc + row;
                if (vec_ok && row + 1 < rows_left) {
                  old[nb][h][mi] = *reinterpret_cast<const double2*>(src);
                } else {
                  old[nb][h][mi].x = src[0];
                  if (row + 1 < rows_left) old[nb][h][mi].y = src[1];
                }
              }
            }
      }
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int mi = 0; mi < MI; ++mi) {
            const int col = (nb0 + nb) * 8 + h, row = mi * 16;
            if (col >= cols_left || row >= rows_left) continue;
            double v0 = p.alpha * acc.c[mi][nb0 + nb][h], v1 = p.alpha * acc.c[mi][nb0 + nb][2 + h];
            if (use_beta) {
              v0 += p.beta * old[nb][h][mi].x;
              v1 += p.beta * old[nb][h][mi].y;
            }
            double* dst = base + col * p.ldc + row;
            if (vec_ok && row + 1 < rows_left) {
              *reinterpret_cast<double2*>(dst) = make_double2(v0, v1);
            } else {
              dst[0] = v0;
              if (row + 1 < rows_left) dst[1] = v1;
            }
          }
    }
  }

  // Element-wise epilogue for tiles that cross the diagonal of a triangular update: only elements inside the
  // stored triangle are read or written.
  static __device__ __forceinline__ void epilogue_masked(const Acc& acc, const GemmArgs<double>& p, double* C,
                                                         int64_t m0, int64_t n0, int warp_m, int warp_n, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const bool use_beta = (p.beta != 0.0);
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
      for (int ni = 0; ni < NI; ++ni)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int64_t row = m0 + warp_m * WTM + mi * 16 + 2 * g + (r >> 1);
          const int64_t col = n0 + warp_n * WTN + ni * 8 + 2 * t + (r & 1);
          if (row < p.m && col < p.n && in_triangle(p.tri, row, col)) {
            double* dst = C + col * p.ldc + row;
            double v = p.alpha * acc.c[mi][ni][r];
            if (use_beta) v += p.beta * *dst;
            *dst = v;
          }
        }
  }
};

// ---------------------------------------------------------------------------------------
// Micro-kernel 2: scalar FMA outer products (FP32 FFMA; also FP64 DFMA).
//
// Both operands are packed into the OC layout (the paper's packed micro-panels: a column of
// A and a row of B are each contiguous), transposing while staging when the source is
// k-contiguous.  Each thread keeps a TM x TN = 8 x 8 accumulator block in registers and per
// k performs the rank-1 update acc += a b^T with a (8 values) and b (8 values) fetched by
// 16-byte shared-memory loads: 64 independent FMAs per outer product.
// A warp is 8 lanes along m by 4 lanes along n, so it covers 64 x 32 of C.
// ---------------------------------------------------------------------------------------
template <typename T_, int BM_, int BN_, int BK_, int WARPS_M, int WARPS_N, bool TA, bool TB, bool PACKED = true,
          int TM_ = 8, int TN_ = 8, bool REGB_ = false>
struct SimtMicro {
  // REGB: a k-contiguous B (not transposed) is transposed through registers (16-byte global loads along k, 4-byte
  // shared-memory stores) instead of by 4-byte cp.async; see GemmKernel::run.
  static constexpr bool REG_TRANSPOSE_B = REGB_ && !TB && sizeof(T_) == 4;
  // k split over a cluster (fp32 packed-pair kernels): the accumulators of a thread as TM/2 * TN 64-bit words
  static constexpr bool HAS_KSPLIT = (sizeof(T_) == 4) && PACKED;
  static constexpr int ACC_WORDS = (TM_ / 2) * TN_;
  using T = T_;
  // fp32 only: PACKED uses the pair instruction fma.rn.f32x2; false keeps scalar FFMA (comparison variant)
  static constexpr bool PAIRS = (sizeof(T_) == 4) && PACKED;
  static constexpr int BM = BM_, BN = BN_, BK = BK_;
  static constexpr int NT = 32 * WARPS_M * WARPS_N;
  static constexpr int VEC = 16 / sizeof(T);
  // per-thread block: 8 x 8 for large problems; 4 x 4 quadruples the warps per tile for small ones
  static constexpr int TM = TM_, TN = TN_;
  static_assert(TM % VEC == 0 && TN % VEC == 0 && TM % 2 == 0, "thread block must be whole 16-byte vectors");
  static constexpr int WTM = 8 * TM, WTN = 4 * TN;
  static_assert(BM == WARPS_M * WTM && BN == WARPS_N * WTN, "CTA tile must be warps x (8 TM x 4 TN)");
  static constexpr Layout LA = OC, LB = OC;
  static constexpr int PA = BM + VEC, PB = BN + VEC;
  static constexpr int A_STAGE = BK * PA, B_STAGE = BK * PB;
  using VT = typename std::conditional<sizeof(T) == 4, float4, double2>::type;

  // Accumulators: scalar c[i][j] for fp64; for fp32 packed row pairs p[i/2][j] = (c[i][j], c[i+1][j]), i even.
  struct AccScalar {
    T c[TM][TN];
  };
  struct AccPairs {
    unsigned long long p[TM / 2][TN];
  };
  using Acc = typename std::conditional<PAIRS, AccPairs, AccScalar>::type;
  static __device__ __forceinline__ unsigned long long get_word(const AccPairs& acc, int w) { return acc.p[w / TN][w % TN]; }
  // acc[w] += b on both halves of a pair (two IEEE fp32 additions)
  static __device__ __forceinline__ void add_word(AccPairs& acc, int w, unsigned long long b) {
    unsigned long long& a = acc.p[w / TN][w % TN];
    float a0, a1, b0, b1;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(a));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(b0), "=f"(b1) : "l"(b));
    a0 = __fadd_rn(a0, b0), a1 = __fadd_rn(a1, b1);
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(a0), "f"(a1));
  }
  // (scalar accumulators are never split: HAS_KSPLIT is false for them)
  static __device__ __forceinline__ unsigned long long get_word(const AccScalar&, int) { return 0ull; }
  static __device__ __forceinline__ void add_word(AccScalar&, int, unsigned long long) {}

  static __device__ __forceinline__ void zero(Acc& acc) {
    if constexpr (PAIRS) {
#pragma unroll
      for (int i = 0; i < TM / 2; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc.p[i][j] = 0ull;
    } else {
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc.c[i][j] = T(0);
    }
  }

  // accumulator element (i, j)
  static __device__ __forceinline__ T get(const Acc& acc, int i, int j) {
    if constexpr (PAIRS) {
      float lo, hi;
      asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc.p[i / 2][j]));
      return (i & 1) ? hi : lo;
    } else {
      return acc.c[i][j];
    }
  }

  // sum of a thread's accumulators (probes keep their result alive through it)
  static __device__ __forceinline__ T checksum(const Acc& acc) {
    T s = T(0);
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) s += get(acc, i, j);
    return s;
  }

  static __device__ __forceinline__ void load_vec(T* dst, const T* src) {
    const VT v = *reinterpret_cast<const VT*>(src);
    if constexpr (sizeof(T) == 4) {
      dst[0] = v.x, dst[1] = v.y, dst[2] = v.z, dst[3] = v.w;
    } else {
      dst[0] = v.x, dst[1] = v.y;
    }
  }

  static __device__ __forceinline__ void compute(Acc& acc, const T* __restrict__ sA, const T* __restrict__ sB,
                                                 int warp_m, int warp_n, int lane) {
    const int lx = lane & 7, ly = lane >> 3;
    const T* pa = sA + warp_m * WTM + lx * VEC;
    const T* pb = sB + warp_n * WTN + ly * VEC;
    if constexpr (PAIRS) {
      // FP32: packed pair multiply-adds (fma.rn.f32x2, two IEEE fp32 FMAs per instruction).  A pair holds two
      // adjacent rows of one column of the accumulator block; a is used pairwise as loaded, b is duplicated
      // into both halves.  32 instructions instead of 64 per outer product: the FP32 pipe stays busy while
      // half of the issue slots are free for the shared-memory loads and the staging code.
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        unsigned long long ap[TM / 2], bd[TN];
#pragma unroll
        for (int gi = 0; gi < TM / VEC; ++gi) {
          const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(pa + kk * PA + gi * 8 * VEC);
          ap[2 * gi] = v.x, ap[2 * gi + 1] = v.y;
        }
#pragma unroll
        for (int gj = 0; gj < TN / VEC; ++gj) {
          const float4 v = *reinterpret_cast<const float4*>(pb + kk * PB + gj * 4 * VEC);
          asm("mov.b64 %0, {%1, %1};" : "=l"(bd[4 * gj + 0]) : "f"(v.x));
          asm("mov.b64 %0, {%1, %1};" : "=l"(bd[4 * gj + 1]) : "f"(v.y));
          asm("mov.b64 %0, {%1, %1};" : "=l"(bd[4 * gj + 2]) : "f"(v.z));
          asm("mov.b64 %0, {%1, %1};" : "=l"(bd[4 * gj + 3]) : "f"(v.w));
        }
#pragma unroll
        for (int ip = 0; ip < TM / 2; ++ip)
#pragma unroll
          for (int j = 0; j < TN; ++j)
            asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc.p[ip][j]) : "l"(ap[ip]), "l"(bd[j]));
      }
    } else {
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        T a[TM], b[TN];
#pragma unroll
        for (int gi = 0; gi < TM / VEC; ++gi) load_vec(a + gi * VEC, pa + kk * PA + gi * 8 * VEC);
#pragma unroll
        for (int gj = 0; gj < TN / VEC; ++gj) load_vec(b + gj * VEC, pb + kk * PB + gj * 4 * VEC);
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc.c[i][j] = fma(a[i], b[j], acc.c[i][j]);
      }
    }
  }

  // C := alpha*acc + beta*C; old C values are fetched in batches of columns before any store of the batch.
  static __device__ __forceinline__ void epilogue(const Acc& acc, const GemmArgs<T>& p, T* C, int64_t m0, int64_t n0,
                                                  int warp_m, int warp_n, int lane) {
    const int lx = lane & 7, ly = lane >> 3;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((p.ldc % VEC) == 0);
    const bool use_beta = (p.beta != T(0));
    constexpr int JB = 2;  // columns per batch: 16 old values in flight
    const int64_t row0 = m0 + warp_m * WTM + lx * VEC;
    const int64_t col0 = n0 + warp_n * WTN + ly * VEC;
#pragma unroll
    for (int j0 = 0; j0 < TN; j0 += JB) {
      T old[JB][TM];
      if (use_beta) {
#pragma unroll
        for (int jb = 0; jb < JB; ++jb) {
          const int j = j0 + jb;
          const int64_t col = col0 + (j / VEC) * 4 * VEC + (j % VEC);
#pragma unroll
          for (int gi = 0; gi < TM / VEC; ++gi) {
            const int64_t row = row0 + gi * 8 * VEC;
#pragma unroll
            for (int e = 0; e < VEC; ++e) old[jb][gi * VEC + e] = T(0);
            if (col < p.n && row < p.m) {
              const T* src = C + col * p.ldc + row;
              if (vec_ok && row + VEC <= p.m) {
                load_vec(&old[jb][gi * VEC], src);
              } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                  if (row + e < p.m) old[jb][gi * VEC + e] = src[e];
              }
            }
          }
        }
      }
#pragma unroll
      for (int jb = 0; jb < JB; ++jb) {
        const int j = j0 + jb;
        const int64_t col = col0 + (j / VEC) * 4 * VEC + (j % VEC);
        if (col >= p.n) continue;
#pragma unroll
        for (int gi = 0; gi < TM / VEC; ++gi) {
          const int64_t row = row0 + gi * 8 * VEC;
          if (row >= p.m) continue;
          T v[VEC];
#pragma unroll
          for (int e = 0; e < VEC; ++e) {
            v[e] = p.alpha * get(acc, gi * VEC + e, j);
            if (use_beta) v[e] += p.beta * old[jb][gi * VEC + e];
          }
          T* dst = C + col * p.ldc + row;
          if (vec_ok && row + VEC <= p.m) {
            VT out;
            if constexpr (sizeof(T) == 4) {
              out = make_float4(v[0], v[1], v[2], v[3]);
            } else {
              out = make_double2(v[0], v[1]);
            }
            *reinterpret_cast<VT*>(dst) = out;
          } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e)
              if (row + e < p.m) dst[e] = v[e];
          }
        }
      }
    }
  }
  // Element-wise epilogue for tiles that cross the diagonal of a triangular update.
  static __device__ __forceinline__ void epilogue_masked(const Acc& acc, const GemmArgs<T>& p, T* C, int64_t m0,
                                                         int64_t n0, int warp_m, int warp_n, int lane) {
    const int lx = lane & 7, ly = lane >> 3;
    const bool use_beta = (p.beta != T(0));
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t col = n0 + warp_n * WTN + (j / VEC) * 4 * VEC + ly * VEC + (j % VEC);
#pragma unroll
      for (int i = 0; i < TM; ++i) {
        const int64_t row = m0 + warp_m * WTM + (i / VEC) * 8 * VEC + lx * VEC + (i % VEC);
        if (row < p.m && col < p.n && in_triangle(p.tri, row, col)) {
          T* dst = C + col * p.ldc + row;
          T v = p.alpha * get(acc, i, j);
          if (use_beta) v += p.beta * *dst;
          *dst = v;
        }
      }
    }
  }
};

// ---------------------------------------------------------------------------------------
// The kernel.  One CTA computes one BM x BN tile of C.
//   ALIGNED: every column of A and B starts on a 16-byte boundary (base pointers 16-byte
//   aligned, leading dimensions multiples of 16/sizeof(T)); otherwise operands are staged
//   element by element.
// ---------------------------------------------------------------------------------------
// ---------------------------------------------------------------------------------------
// Drain through shared memory, for beta == 1 (C := C + alpha op(A) op(B), the trailing update of a factorisation)
// and beta == 0.  A tile that lies wholly inside C (and inside the stored triangle of a triangular update) and
// whose columns of C are 16-byte aligned leaves as alpha * acc through shared memory that the operand ring no
// longer needs, and one thread per column issues a bulk copy: a reduction that ADDS the column to C in memory
// (beta == 1), or a plain store (beta == 0).  No thread loads an old value of C, waits for one, or holds its
// accumulators while stores drain.  The arithmetic is the ordinary epilogue's (alpha * acc rounded; with beta = 1
// one addition to the old value), so the bits are the same.  Used by the TMA-staged kernels; in the cp.async fp32
// kernels it was measured and changed nothing (16384^2 x 64: 42.9 against 43.4 TFLOP/s; their drain is not what
// they wait for), and the cp.async fp64 64 x 64 kernel has no register to spare for it.
// ---------------------------------------------------------------------------------------
template <class Micro>
__device__ __forceinline__ bool tile_added_in_memory(const GemmArgs<typename Micro::T>& p, const typename Micro::T* C,
                                                     int64_t m0, int64_t n0) {
  using T = typename Micro::T;
  return (p.beta == T(1) || p.beta == T(0)) && !tile_crosses_diagonal(p.tri, m0, n0, Micro::BM, Micro::BN) && m0 + Micro::BM <= p.m &&
         n0 + Micro::BN <= p.n && (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (p.ldc % (16 / (int)sizeof(T))) == 0;
}
// Every thread of the CTA calls this after its last read of the ring; sC is the ring's first byte.
template <class Micro>
__device__ __forceinline__ void drain_by_reduction(const typename Micro::Acc& acc, const GemmArgs<typename Micro::T>& p,
                                                   typename Micro::T* C, int64_t m0, int64_t n0,
                                                   typename Micro::T* sC, int warp_m, int warp_n, int lane) {
  using T = typename Micro::T;
  __syncthreads();  // every warp has finished reading the ring
  Micro::stage_tile(acc, p.alpha, sC, warp_m, warp_n, lane);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // these writes are read by the async proxy
  __syncthreads();
  for (int c = threadIdx.x; c < Micro::BN; c += Micro::NT) {
    if (p.beta == T(0))  // nothing to add to: a plain bulk store
      bulk_store(C + (n0 + c) * p.ldc + m0, sC + c * Micro::PC, (uint32_t)(Micro::BM * sizeof(T)));
    else
      bulk_reduce_add(C + (n0 + c) * p.ldc + m0, sC + c * Micro::PC, (uint32_t)(Micro::BM * sizeof(T)));
  }
  bulk_commit();
  bulk_wait_read_all();  // the shared memory must outlive the reads of the reductions
}

template <class Micro, int STAGES, bool TA, bool TB, bool ALIGNED>
struct GemmKernel {
  using T = typename Micro::T;
  static constexpr int BM = Micro::BM, BN = Micro::BN, BK = Micro::BK, NT = Micro::NT;
  static constexpr Layout SRC_A = TA ? KC : OC;
  static constexpr Layout SRC_B = TB ? OC : KC;
  static constexpr int VEC = ALIGNED ? (16 / (int)sizeof(T)) : 1;
  using StageA = Stager<T, BM, BK, NT, SRC_A, Micro::LA, VEC, Micro::PA>;
  using StageB = Stager<T, BN, BK, NT, SRC_B, Micro::LB, VEC, Micro::PB>;
  static constexpr size_t SMEM_BYTES = (size_t)STAGES * (Micro::A_STAGE + Micro::B_STAGE) * sizeof(T);
  // k split over a cluster: the micro-kernel supports it and the ring can hold a CTA's accumulators
  static constexpr bool KSPLIT_OK = Micro::HAS_KSPLIT && SMEM_BYTES >= (size_t)BM * BN * sizeof(T);

  static __device__ __forceinline__ void run(const GemmArgs<T>& p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* sA = reinterpret_cast<T*>(smem_raw);
    T* sB = sA + STAGES * Micro::A_STAGE;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int warp_m = warp % (BM / Micro::WTM), warp_n = warp / (BM / Micro::WTM);

    int tm, tn;
    tile_coords(blockIdx.x, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
    const int64_t m0 = (int64_t)tm * BM, n0 = (int64_t)tn * BN;
    if (tile_outside_triangle(p.tri, m0, n0, BM, BN)) return;  // triangular update: nothing of this tile is stored
    const int m_valid = (int)min((int64_t)BM, p.m - m0), n_valid = (int)min((int64_t)BN, p.n - n0);

    // element (m0, 0) of op(A) and (0, n0) of op(B) of problem blockIdx.y of a strided batch
    const T* gA = p.A + (int64_t)blockIdx.y * p.batch_a + (TA ? m0 * p.lda : m0);
    const T* gB = p.B + (int64_t)blockIdx.y * p.batch_b + (TB ? n0 : n0 * p.ldb);
    const int64_t stepA = TA ? (int64_t)BK : (int64_t)BK * p.lda;  // advance by BK along k
    const int64_t stepB = TB ? (int64_t)BK * p.ldb : (int64_t)BK;

    const int KT_all = (int)((p.k + BK - 1) / BK);
    const bool a_inside = (m_valid == BM), b_inside = (n_valid == BN);
    // k split over a cluster: this CTA takes slabs [kt0, kt1) of the tile (possibly none)
    int kt0 = 0, kt1 = KT_all;
    if constexpr (KSPLIT_OK) {
      if (p.ksplit > 1) {
        const int per = (KT_all + p.ksplit - 1) / p.ksplit;
        kt0 = min(KT_all, (int)blockIdx.z * per), kt1 = min(KT_all, kt0 + per);
        gA += (int64_t)kt0 * stepA;
        gB += (int64_t)kt0 * stepB;
      }
    }
    const int KT = kt1 - kt0;
    // valid k-entries of this CTA's last slab
    const int k_tail = (kt1 == KT_all) ? (int)(p.k - (int64_t)(KT_all - 1) * BK) : BK;

    StageA stA;
    StageB stB;
    stA.init(gA, p.lda, tid);
    stB.init(gB, p.ldb, tid);

    // beta != 0: pull this tile's old C values towards L2 now, so that the epilogue's loads overlap the k-loop
    // instead of paying the DRAM latency after it (this matters when k is only a few slabs).
    if (p.beta != T(0) && (!KSPLIT_OK || blockIdx.z == 0)) {
      constexpr int LINE = 128 / (int)sizeof(T);   // elements per 128-byte line
      constexpr int LPC = (BM + LINE - 1) / LINE;  // lines per tile column
      for (int c = tid; c < BN * LPC; c += NT) {
        const int col = c / LPC, row = (c % LPC) * LINE;
        if (col < n_valid && row < m_valid) {
          const T* ptr = p.C + (int64_t)blockIdx.y * p.batch_c + (n0 + col) * p.ldc + m0 + row;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
        }
      }
    }

    // stage slab kt (slabs are staged in increasing order, so the running pointers follow along)
    auto stage = [&](int kt, int slot) {
      const int k_valid = (kt == KT - 1) ? k_tail : BK;
      T* dA = sA + slot * Micro::A_STAGE;
      T* dB = sB + slot * Micro::B_STAGE;
      if (k_valid == BK) {
        if (a_inside) {
          stA.load_fast(dA, p.lda, tid);
        } else {
          stA.load_edge(dA, p.lda, m_valid, tid);
        }
        if (b_inside) {
          stB.load_fast(dB, p.ldb, tid);
        } else {
          stB.load_edge(dB, p.ldb, n_valid, tid);
        }
      } else {
        StageA::load_general(dA, gA + kt * stepA, p.lda, m_valid, k_valid, tid);
        StageB::load_general(dB, gB + kt * stepB, p.ldb, n_valid, k_valid, tid);
      }
      stA.advance(p.lda);
      stB.advance(p.ldb);
    };

    // ramp-up: fill STAGES-1 slots (the first of the paper's three stages of the k-loop)
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
      if (s < KT) stage(s, s);
      cp_async_commit();
    }

    typename Micro::Acc acc;
    Micro::zero(acc);

    // Transposition of a k-contiguous B through registers (fp32 FMA kernels, 16-byte aligned columns, full
    // interior slabs): while slab kt is being multiplied, the thread's share of slab kt+STAGES-1 travels from
    // global memory into registers in 16-byte pieces along k; after the multiply-adds it is written to the free
    // ring slot element by element, transposed.  A pair of lanes reads one 32-byte sector of a column, a warp 16
    // columns; the stores of a warp fall into 32 different banks (pitch = 4 mod 32 words).  The next CTA-wide
    // barrier publishes the slot, which is not read before the iteration after it.
    constexpr bool REGB = Micro::REG_TRANSPOSE_B && ALIGNED;
    constexpr int NBR = REGB ? (BN * BK / 4) / NT : 1;
    static_assert(!REGB || ((BN * BK / 4) % NT == 0 && (BK / 4) % 2 == 0 && NT % 2 == 0 && (BN % (NT / 2) == 0 || (NT / 2) % BN == 0)),
                  "register transposition geometry");
    float4 breg[NBR];

    // steady state: wait for slab kt, refill the slot freed in the previous iteration, compute
    int slot = 0, fill = STAGES - 1;
    for (int kt = 0; kt < KT; ++kt) {
      cp_async_wait<STAGES - 2>();
      __syncthreads();
      const int next = kt + STAGES - 1;
      bool by_regs = false;
      if constexpr (REGB) by_regs = (next < KT) && b_inside && (next != KT - 1 || k_tail == BK);
      if (by_regs) {
        if constexpr (REGB) {
          T* dA = sA + fill * Micro::A_STAGE;
          if (a_inside) {
            stA.load_fast(dA, p.lda, tid);
          } else {
            stA.load_edge(dA, p.lda, m_valid, tid);
          }
          stA.advance(p.lda);
          stB.advance(p.ldb);
          const T* gBn = gB + (int64_t)next * BK;
#pragma unroll
          for (int it = 0; it < NBR; ++it) {
            const int c = tid + it * NT;
            const int n = (c >> 1) % BN, kq = ((c >> 1) / BN) * 2 + (c & 1);
            breg[it] = *reinterpret_cast<const float4*>(gBn + (int64_t)n * p.ldb + kq * 4);
          }
        }
      } else if (next < KT) {
        stage(next, fill);
      }
      cp_async_commit();
      Micro::compute(acc, sA + slot * Micro::A_STAGE, sB + slot * Micro::B_STAGE, warp_m, warp_n, lane);
      if constexpr (REGB) {
        if (by_regs) {
          T* dB = sB + fill * Micro::B_STAGE;
#pragma unroll
          for (int it = 0; it < NBR; ++it) {
            const int c = tid + it * NT;
            const int n = (c >> 1) % BN, kq = ((c >> 1) / BN) * 2 + (c & 1);
            T* d = dB + (kq * 4) * Micro::PB + n;
            d[0] = breg[it].x, d[Micro::PB] = breg[it].y, d[2 * Micro::PB] = breg[it].z, d[3 * Micro::PB] = breg[it].w;
          }
        }
      }
      slot = (slot + 1 == STAGES) ? 0 : slot + 1;
      fill = (fill + 1 == STAGES) ? 0 : fill + 1;
    }
    cp_async_wait<0>();

    // k split: the partial sums of ranks 1 .. ksplit-1 go through their (now idle) rings; rank 0 adds them in rank
    // order, element by element, so the result does not depend on timing.  Every thread of every CTA of the
    // cluster passes both cluster barriers: a split launch has no early exit (tri == 0).
    if constexpr (KSPLIT_OK) {
      if (p.ksplit > 1) {
        unsigned long long* sAcc = reinterpret_cast<unsigned long long*>(smem_raw);
        __syncthreads();  // every warp has finished reading the ring
        if (blockIdx.z != 0) {
#pragma unroll
          for (int w = 0; w < Micro::ACC_WORDS; ++w) sAcc[w * NT + tid] = Micro::get_word(acc, w);
        }
        cluster_sync_all();  // partial sums are visible across the cluster
        if (blockIdx.z == 0) {
          for (int r = 1; r < p.ksplit; ++r) {
            const uint32_t remote = cluster_map_shared(smem_u32(sAcc), (uint32_t)r);
#pragma unroll
            for (int w = 0; w < Micro::ACC_WORDS; ++w)
              Micro::add_word(acc, w, ld_cluster_b64(remote + (uint32_t)((w * NT + tid) * 8)));
          }
        }
        cluster_sync_all();  // rank 0 has read everything: the other CTAs may leave
        if (blockIdx.z != 0) return;
      }
    }

    // drain: fused alpha/beta epilogue
    T* Cb = p.C + (int64_t)blockIdx.y * p.batch_c;
    if (tile_crosses_diagonal(p.tri, m0, n0, BM, BN)) {
      Micro::epilogue_masked(acc, p, Cb, m0, n0, warp_m, warp_n, lane);
    } else {
      Micro::epilogue(acc, p, Cb, m0, n0, warp_m, warp_n, lane);
    }
  }
};

template <class Kernel, int MIN_CTAS>
__global__ void __launch_bounds__(Kernel::NT, MIN_CTAS) gemm_kernel(const GemmArgs<typename Kernel::T> p) {
  Kernel::run(p);
}

// C := beta*C for the quick-return cases (alpha == 0 or k == 0); beta == 0 stores zeros
// without reading C.
template <typename T>
__global__ void scale_kernel(int64_t m, int64_t n, T beta, T* C, int64_t ldc) {
  const int64_t total = m * n;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
       idx += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = idx % m, j = idx / m;
    T* c = C + i + j * ldc;
    *c = (beta == T(0)) ? T(0) : beta * *c;
  }
}

}  // namespace b2
