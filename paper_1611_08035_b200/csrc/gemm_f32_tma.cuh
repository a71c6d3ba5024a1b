// FP32 packed-pair micro-kernels fed by the tensor memory accelerator.
//
// The cp.async-staged fp32 kernels spend 5 to 8 instructions per rank-1 update on staging (copy instructions, their
// 64-bit address arithmetic, the barrier), and every one of them takes an issue slot from the pair instructions,
// which at peak fill the dispatch port by themselves.  Here one thread hands whole operand slabs to the TMA and
// the multiplying warps run the bare loop: fragment loads and pair instructions, one mbarrier wait and one arrive
// per slab.
//
// No copy can transpose, so each operand sits in shared memory the way it sits in global memory, and the loop
// adapts to the layout instead (the paper packs both operands into the order its micro-kernel reads; with the TMA
// the micro-kernel reads the order the operands have):
//   * an operand whose C index is contiguous (A not transposed: m; B transposed: n) arrives as BK lines of the
//     tile's extent; a lane reads 4 consecutive values of one k with a 16-byte load, as the cp.async kernels do;
//   * a k-contiguous operand (A transposed, B not transposed) arrives as one 64-byte line of 16 k per row or
//     column of the tile, the 16-byte pieces of each line permuted by the TMA's 64-byte swizzle; a lane reads
//     4 consecutive k of ONE row/column with a 16-byte load, and the lanes of a warp take consecutive
//     rows/columns, which the swizzle spreads over all banks.  The lane's rows are then lx, lx + 8, ... instead
//     of groups of four neighbours.
// The pair instruction multiplies two values of one operand by one value of the other.  The paired operand must
// have its two values in neighbouring registers:
//   * A with m contiguous: pairs of neighbouring rows, b in both halves (the form the cp.async kernels use);
//   * A k-contiguous, B with n contiguous: pairs of neighbouring columns, a in both halves;
//   * both k-contiguous: no operand has two values of one k in neighbouring registers.  Pairing neighbouring k
//     instead (an element of C kept as two partial sums, even and odd k, added at the end) doubles the accumulator
//     registers for the same block; built and measured at 45 TFLOP/s against 54.7 for the cp.async kernel at
//     8192^3, it is not kept, and the launcher declines that case.
#pragma once
#include "gemm_tma.cuh"

namespace b2 {

template <int TM_, int TN_, int WARPS_M, int WARPS_N, bool TA, bool TB>
struct SimtTmaMicro {
  using T = float;
  static constexpr int TM = TM_, TN = TN_;
  static constexpr int WTM = 8 * TM, WTN = 4 * TN;
  static constexpr int BM = WARPS_M * WTM, BN = WARPS_N * WTN, BK = 16;
  static constexpr int NT = 32 * WARPS_M * WARPS_N;
  static constexpr bool A_KC = TA, B_KC = !TB;  // k-contiguous in memory, hence in shared memory
  // box inner extents (the kernel derives the outer ones): a 64-byte line of k, or the tile's whole extent
  static constexpr int PA = A_KC ? BK : BM, PB = B_KC ? BK : BN;
  static constexpr int A_STAGE = BM * BK, B_STAGE = BN * BK;
  static constexpr bool SWIZZLE_A = A_KC, SWIZZLE_B = B_KC;
  static_assert(!(A_KC && B_KC), "one operand must have its C index contiguous");
  static constexpr int PAIR_ROWS = 0, PAIR_COLS = 1;
  static constexpr int PAIRING = !A_KC ? PAIR_ROWS : PAIR_COLS;
  static constexpr int WORDS = TM * TN / 2;
  static_assert(TM % 4 == 0 && TN % 4 == 0, "blocks are built from 16-byte loads");
  static_assert(BM <= 256 && BN <= 256, "a TMA box is at most 256 elements wide");

  struct Acc {
    unsigned long long p[WORDS];
  };
  static __device__ __forceinline__ void zero(Acc& acc) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) acc.p[w] = 0ull;
  }

  // rows / columns of the warp's block that a lane owns (i < TM, j < TN)
  static __device__ __forceinline__ int row_of(int i, int lx) {
    return A_KC ? lx + 8 * i : (i / 4) * 32 + lx * 4 + (i % 4);
  }
  static __device__ __forceinline__ int col_of(int j, int ly) {
    return B_KC ? ly + 4 * j : (j / 4) * 16 + ly * 4 + (j % 4);
  }

  // element (i, j) of the lane's block
  static __device__ __forceinline__ float get(const Acc& acc, int i, int j) {
    float lo, hi;
    if constexpr (PAIRING == PAIR_ROWS) {
      asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc.p[(i / 2) * TN + j]));
      return (i & 1) ? hi : lo;
    } else {
      asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc.p[i * (TN / 2) + j / 2]));
      return (j & 1) ? hi : lo;
    }
  }

  static __device__ __forceinline__ unsigned long long both_halves(float v) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(v));
    return r;
  }
  static __device__ __forceinline__ void fma2(unsigned long long& c, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(c) : "l"(a), "l"(b));
  }
  static __device__ __forceinline__ float pick(const float4& v, int kk) {
    return kk == 0 ? v.x : (kk == 1 ? v.y : (kk == 2 ? v.z : v.w));
  }

  // One 16-deep slab.  sA, sB: the stage's two boxes (1024-byte aligned).
  static __device__ __forceinline__ void compute(Acc& acc, const float* __restrict__ sA, const float* __restrict__ sB,
                                                 int warp_m, int warp_n, int lane) {
    const int lx = lane & 7, ly = lane >> 3;
    // k-contiguous boxes: row r holds its piece q (k = 4q .. 4q+3) at piece index q ^ ((r >> 1) & 3).  The warp's
    // first row is a multiple of 8 and a lane's rows are lx + 8 i (columns: ly + 4 j), so the XOR term is
    // (lx >> 1) for A and (ly >> 1) | ((j & 1) << 1) for B: one lane-dependent part, one compile-time part.
    const float* pa = A_KC ? sA + (warp_m * WTM + lx) * BK : sA + warp_m * WTM + lx * 4;
    const float* pb = B_KC ? sB + (warp_n * WTN + ly) * BK : sB + warp_n * WTN + ly * 4;
    const int swa = (lx >> 1) & 3;
    // piece c of a lane with (ly >> 1) set sits at c ^ 1: four floats further for even c, four back for odd c
    const float* pb_even = pb + 4 * (ly >> 1);
    const float* pb_odd = pb - 4 * (ly >> 1);

    if constexpr (PAIRING == PAIR_ROWS && !B_KC) {
      // both operands with the C index contiguous: per k, TM/4 + TN/4 loads and TM*TN/2 pair instructions
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        unsigned long long ap[TM / 2], bd[TN];
#pragma unroll
        for (int gi = 0; gi < TM / 4; ++gi) {
          const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(pa + kk * BM + gi * 32);
          ap[2 * gi] = v.x, ap[2 * gi + 1] = v.y;
        }
#pragma unroll
        for (int gj = 0; gj < TN / 4; ++gj) {
          const float4 v = *reinterpret_cast<const float4*>(pb + kk * BN + gj * 16);
          bd[4 * gj] = both_halves(v.x), bd[4 * gj + 1] = both_halves(v.y);
          bd[4 * gj + 2] = both_halves(v.z), bd[4 * gj + 3] = both_halves(v.w);
        }
#pragma unroll
        for (int ip = 0; ip < TM / 2; ++ip)
#pragma unroll
          for (int j = 0; j < TN; ++j) fma2(acc.p[ip * TN + j], ap[ip], bd[j]);
      }
    } else if constexpr (PAIRING == PAIR_ROWS && B_KC) {
      // A with m contiguous, B k-contiguous: four k of every column of b at a time
#pragma unroll
      for (int q = 0; q < BK / 4; ++q) {
        float4 b4[TN];
#pragma unroll
        for (int j = 0; j < TN; ++j) {
          const int c = q ^ ((j & 1) << 1);  // compile time; the lane's bit flips the piece's lowest bit
          b4[j] = *reinterpret_cast<const float4*>(((c & 1) ? pb_odd : pb_even) + 4 * j * BK + c * 4);
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          unsigned long long ap[TM / 2];
#pragma unroll
          for (int gi = 0; gi < TM / 4; ++gi) {
            const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(pa + (4 * q + kk) * BM + gi * 32);
            ap[2 * gi] = v.x, ap[2 * gi + 1] = v.y;
          }
          unsigned long long bd[TN];
#pragma unroll
          for (int j = 0; j < TN; ++j) bd[j] = both_halves(pick(b4[j], kk));
#pragma unroll
          for (int ip = 0; ip < TM / 2; ++ip)
#pragma unroll
            for (int j = 0; j < TN; ++j) fma2(acc.p[ip * TN + j], ap[ip], bd[j]);
        }
      }
    } else {
      // A k-contiguous, B with n contiguous: pairs of neighbouring columns, a in both halves
#pragma unroll
      for (int q = 0; q < BK / 4; ++q) {
        float4 a4[TM];
#pragma unroll
        for (int i = 0; i < TM; ++i) a4[i] = *reinterpret_cast<const float4*>(pa + 8 * i * BK + ((q ^ swa) * 4));
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          unsigned long long bp[TN / 2];
#pragma unroll
          for (int gj = 0; gj < TN / 4; ++gj) {
            const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(pb + (4 * q + kk) * BN + gj * 16);
            bp[2 * gj] = v.x, bp[2 * gj + 1] = v.y;
          }
#pragma unroll
          for (int i = 0; i < TM; ++i) {
            const unsigned long long ad = both_halves(pick(a4[i], kk));
#pragma unroll
            for (int jp = 0; jp < TN / 2; ++jp) fma2(acc.p[i * (TN / 2) + jp], ad, bp[jp]);
          }
        }
      }
    }
  }

  // alpha * acc into a column-major tile in shared memory (column pitch PC, 16-byte aligned columns)
  static constexpr int PC = BM + 4;
  static __device__ __forceinline__ void stage_tile(const Acc& acc, float alpha, float* sC, int warp_m, int warp_n,
                                                    int lane) {
    const int lx = lane & 7, ly = lane >> 3;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      float* col = sC + (warp_n * WTN + col_of(j, ly)) * PC + warp_m * WTM;
#pragma unroll
      for (int g = 0; g < TM / 4; ++g) {
        if constexpr (!A_KC) {  // four neighbouring rows
          *reinterpret_cast<float4*>(col + row_of(4 * g, lx)) =
              make_float4(alpha * get(acc, 4 * g, j), alpha * get(acc, 4 * g + 1, j), alpha * get(acc, 4 * g + 2, j),
                          alpha * get(acc, 4 * g + 3, j));
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) col[row_of(4 * g + e, lx)] = alpha * get(acc, 4 * g + e, j);
        }
      }
    }
  }

  // C := alpha*acc + beta*C on the lane's block, column by column; rows >= m and columns >= n are skipped.
  static __device__ __forceinline__ void store(const Acc& acc, const GemmArgs<float>& p, float* C, int64_t m0,
                                               int64_t n0, int warp_m, int warp_n, int lane) {
    const int lx = lane & 7, ly = lane >> 3;
    const bool use_beta = (p.beta != 0.0f);
    const bool vec_ok = !A_KC && ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && ((p.ldc & 3) == 0);
    const int64_t rbase = m0 + warp_m * WTM, cbase = n0 + warp_n * WTN;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t col = cbase + col_of(j, ly);
      if (col >= p.n) continue;
      float* ccol = C + col * p.ldc;
      float old[TM];
      if (use_beta) {
#pragma unroll
        for (int g = 0; g < TM / 4; ++g) {
          const int64_t row = rbase + row_of(4 * g, lx);
          if (vec_ok && row + 4 <= p.m) {
            const float4 v = *reinterpret_cast<const float4*>(ccol + row);
            old[4 * g] = v.x, old[4 * g + 1] = v.y, old[4 * g + 2] = v.z, old[4 * g + 3] = v.w;
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int64_t r = rbase + row_of(4 * g + e, lx);
              old[4 * g + e] = r < p.m ? ccol[r] : 0.0f;
            }
          }
        }
      }
#pragma unroll
      for (int g = 0; g < TM / 4; ++g) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[e] = p.alpha * get(acc, 4 * g + e, j);
          if (use_beta) v[e] += p.beta * old[4 * g + e];
        }
        const int64_t row = rbase + row_of(4 * g, lx);
        if (vec_ok && row + 4 <= p.m) {
          *reinterpret_cast<float4*>(ccol + row) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int64_t r = rbase + row_of(4 * g + e, lx);
            if (r < p.m) ccol[r] = v[e];
          }
        }
      }
    }
  }
  static __device__ __forceinline__ void epilogue(const Acc& acc, const GemmArgs<float>& p, float* C, int64_t m0,
                                                  int64_t n0, int warp_m, int warp_n, int lane) {
    store(acc, p, C, m0, n0, warp_m, warp_n, lane);
  }
  // triangular updates are declined by the launcher, so no tile ever crosses a diagonal
  static __device__ __forceinline__ void epilogue_masked(const Acc& acc, const GemmArgs<float>& p, float* C, int64_t m0,
                                                         int64_t n0, int warp_m, int warp_n, int lane) {
    store(acc, p, C, m0, n0, warp_m, warp_n, lane);
  }
};

}  // namespace b2
