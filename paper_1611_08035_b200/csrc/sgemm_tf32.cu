// fp32 GEMM on the 5th-generation tensor cores in TF32 (tcgen05.mma kind::tf32, accumulator in tensor
// memory), reported separately from b2_sgemm because TF32 changes results: b2_sgemm_tf32x1 rounds both
// operands to TF32 (10 mantissa bits), b2_sgemm_tf32x3 splits each operand into a TF32 head and tail and adds
// the three leading products, which brings the result back to fp32 accuracy.  The paper has no counterpart
// (its kernels are FP64 SIMD); the loop structure is the same sum of rank-k updates over packed panels.
//
// Two steps, both on the caller's stream:
//   1. pack (the paper's packing step, Section 2.1, made explicit): op(A) and op(B) are written to the
//      workspace as K-major panels P[i][p] (p contiguous, zero-padded to a multiple of 32), rounded to TF32
//      with cvt.rna; for the 3-term variant the panels are [hi | hi | lo] for A and [hi | lo | hi] for B, so
//      that one TF32 GEMM over the concatenated k computes hi*hi + hi*lo + lo*hi.
//   2. multiply: one CTA per 128 x 128 tile of C.  A producer thread streams 128 x 32 boxes of both panels
//      into a 6-stage shared-memory ring with TMA (128-byte swizzle), an issuing thread runs
//      tcgen05.mma (M = 128, N = 128, K = 8 per instruction) on the ring with the 128 x 128 fp32
//      accumulator in tensor memory, tcgen05.commit frees ring slots and signals the end, and all four warps
//      then read the accumulator with tcgen05.ld and apply alpha/beta.
// Every mbarrier wait is bounded; on a time-out the status word is set (b2_device_status) and the CTA leaves
// through the common exit that frees its tensor memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "b2gemm.h"
#include "entry.h"
#include "gemm_tma.cuh"

namespace b2 {
namespace {

constexpr int TBM = 128, TBK = 32, UMMA_K = 8;
constexpr uint32_t STAGE_A_BYTES = TBM * TBK * 4;
// Tile width (TBN) and ring depth: 128 x 256 tiles with 4 stages halve the shared-memory bytes read per
// multiply-add (the tensor pipe reads A and B from shared memory for every instruction); 128 x 128 tiles with 6
// stages serve narrow problems.  Either ring is 192 KB; the 2-stage ring of the 128 x 256 tile (96 KB) lets two
// CTAs share an SM.
template <int TBN, int TSTAGES>
struct Tf32Cfg {
  static constexpr uint32_t STAGE_B_BYTES = TBN * TBK * 4;
  static constexpr uint32_t RING_BYTES = TSTAGES * (STAGE_A_BYTES + STAGE_B_BYTES);
  static constexpr size_t SMEM_BYTES = RING_BYTES + 1024 /* alignment slack */ + 256 /* barriers, tmem address */;
};

__device__ int g_tf32_status = 0;

// ---- packing ----------------------------------------------------------------------------------
__device__ __forceinline__ float tf32_rna(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

// P[i][p] for i < rows, p < kpad (pitch = terms*kpad floats): element (i, p) of op(X) rounded to TF32, zero for
// p >= k.  x_is_k_contiguous: op(X)(i, p) = X[p + i*ld], else X[i + p*ld].  For terms == 3 the three column blocks
// hold (hi, hi, lo) when lo_last, (hi, lo, hi) otherwise.
// 64 x 64 tile per CTA of 256 threads, 16-byte loads along whichever index is contiguous in the source (when base
// and leading dimension allow) and 16-byte stores along p: the pass is HBM-bound, so what matters is bytes in flight.
template <bool K_CONTIG>
__global__ void __launch_bounds__(256)
    tf32_pack_kernel(const float* __restrict__ X, int64_t ld, int64_t rows, int64_t k, int64_t kpad, int terms,
                     bool lo_last, float* __restrict__ P) {
  constexpr int TP = 64;
  __shared__ float tile[TP][TP + 1];  // tile[i][p]
  const int64_t i0 = (int64_t)blockIdx.y * TP, p0 = (int64_t)blockIdx.x * TP;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // 16 x 16
  const int64_t pitch = (int64_t)terms * kpad;
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(X) & 15) == 0) && (ld % 4 == 0);
  // c = index along the source's contiguous direction (p when K_CONTIG, else i), s = the other one
  const int64_t c_base = K_CONTIG ? p0 : i0, s_base = K_CONTIG ? i0 : p0;
  const int64_t c_end = K_CONTIG ? k : rows, s_end = K_CONTIG ? rows : k;
#pragma unroll
  for (int it = 0; it < TP / 16; ++it) {
    const int sl = ty + it * 16, cl = tx * 4;
    const int64_t sg = s_base + sl, cg = c_base + cl;
    float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (sg < s_end) {
      const float* src = X + cg + sg * ld;
      if (vec_ok && cg + 3 < c_end) {
        const float4 q = *reinterpret_cast<const float4*>(src);
        v[0] = q.x, v[1] = q.y, v[2] = q.z, v[3] = q.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (cg + e < c_end) v[e] = src[e];
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (K_CONTIG) tile[sl][cl + e] = v[e]; else tile[cl + e][sl] = v[e];
    }
  }
  __syncthreads();
#pragma unroll
  for (int it = 0; it < TP / 16; ++it) {
    const int r = ty + it * 16;
    const int64_t i = i0 + r, p = p0 + tx * 4;
    if (i >= rows || p >= kpad) continue;  // kpad is a multiple of 32: a group of four is inside or outside as a whole
    float hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float x = tile[r][tx * 4 + e];
      hi[e] = tf32_rna(x);
      lo[e] = tf32_rna(x - hi[e]);
    }
    float* row = P + i * pitch + p;
    const float4 vh = make_float4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<float4*>(row) = vh;
    if (terms == 3) {
      const float4 vl = make_float4(lo[0], lo[1], lo[2], lo[3]);
      *reinterpret_cast<float4*>(row + kpad) = lo_last ? vh : vl;
      *reinterpret_cast<float4*>(row + 2 * kpad) = lo_last ? vl : vh;
    }
  }
}

// ---- tcgen05 helpers ---------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem], TF32 inputs, fp32 accumulate; accumulate == 0 overwrites D.
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival when all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 16 consecutive accumulator columns of this lane's row (32 lanes x 32 bits, 16 repetitions); the values are
// defined only after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// The registers pass through the wait as read-write operands, so that no use of them is scheduled before it.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&a)[16], uint32_t (&b)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                 "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                 "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                 "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
               :
               : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes (32 floats) with the
// 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset), the leading byte offset is not
// used by swizzled K-major layouts, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;            // leading byte offset (16 bytes, ignored)
  d |= (uint64_t)(1024 >> 4) << 32;  // stride byte offset
  d |= (uint64_t)1 << 46;            // version
  d |= (uint64_t)2 << 61;            // 128-byte swizzle
  return d;
}
// Instruction descriptor: fp32 accumulator, TF32 A and B, both K-major, N and M of the instruction.
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int m, int n) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// 2-D box with the 128-byte swizzle (same primitive as tma_load_2d; the swizzle lives in the tensor map)
struct Tf32Args {
  int64_t m, n;
  int kt;  // number of 32-wide k slabs of the packed panels
  float alpha, beta;
  float* C;
  int64_t ldc;
  int tiles_m;
  int* status;
};

template <int TBN, int TSTAGES, int MINB = 1>
__global__ void __launch_bounds__(128, MINB)
    sgemm_tf32_kernel(const Tf32Args p, const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB) {
  constexpr uint32_t STAGE_B_BYTES = Tf32Cfg<TBN, TSTAGES>::STAGE_B_BYTES;
  constexpr uint32_t RING_BYTES = Tf32Cfg<TBN, TSTAGES>::RING_BYTES;
  extern __shared__ unsigned char tf32_smem_raw[];
  const uint32_t raw = smem_u32(tf32_smem_raw);
  unsigned char* ring = tf32_smem_raw + (((raw + 1023u) & ~1023u) - raw);  // 1024-byte aligned for the swizzle
  unsigned char* sA = ring;
  unsigned char* sB = ring + TSTAGES * STAGE_A_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(ring + RING_BYTES);
  uint64_t* empty = full + TSTAGES;
  uint64_t* accum = empty + TSTAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tm = blockIdx.x % p.tiles_m, tn = blockIdx.x / p.tiles_m;
  const int64_t m0 = (int64_t)tm * TBM, n0 = (int64_t)tn * TBN;
  const int KT = p.kt;

  if (tid == 0) {
    for (int s = 0; s < TSTAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(accum, 1);
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, TBN);  // TBN columns x 128 lanes of fp32
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  bool ok = true;
  bool committed = false;  // issuing thread: the accumulator's completion has been committed to `accum`
  if (warp == 0 && lane == 0) {
    // ---- producer: TMA boxes of 32 (k) x 128 rows of both panels
    int issued = 0;
    for (int kt = 0; kt < KT && ok; ++kt) {
      const int s = kt % TSTAGES, r = kt / TSTAGES;
      if (r > 0 && !mbar_wait_bounded(&empty[s], (uint32_t)((r - 1) & 1))) {
        ok = false;
        break;
      }
      mbar_arrive_expect_tx(&full[s], STAGE_A_BYTES + STAGE_B_BYTES);
      tma_load_2d(sA + s * STAGE_A_BYTES, &mapA, kt * TBK, (int)m0, &full[s]);
      tma_load_2d(sB + s * STAGE_B_BYTES, &mapB, kt * TBK, (int)n0, &full[s]);
      issued = kt + 1;
    }
    if (!ok) {
      atomicExch(p.status, (int)B2_ERR_TIMEOUT);
      // let the copies still in flight land: the latest fill of every slot
      for (int s = 0; s < TSTAGES; ++s) {
        const int last = ((issued - 1 - s) / TSTAGES) * TSTAGES + s;  // last slab that went to slot s
        if (issued > s && last >= 0)
          (void)mbar_wait_bounded(&full[s], (uint32_t)((last / TSTAGES) & 1), kDrainLimitNs);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- issuer: four K = 8 instructions per slab, accumulator in tensor memory
    constexpr uint32_t idesc = umma_idesc_tf32(TBM, TBN);
    for (int kt = 0; kt < KT; ++kt) {
      const int s = kt % TSTAGES, r = kt / TSTAGES;
      if (!mbar_wait_bounded(&full[s], (uint32_t)(r & 1))) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t a0 = smem_u32(sA + s * STAGE_A_BYTES), b0 = smem_u32(sB + s * STAGE_B_BYTES);
#pragma unroll
      for (int j = 0; j < TBK / UMMA_K; ++j) {
        const uint64_t da = umma_desc_k_major_sw128(a0 + j * UMMA_K * 4);
        const uint64_t db = umma_desc_k_major_sw128(b0 + j * UMMA_K * 4);
        umma_tf32(tmem_d, da, db, idesc, (kt | j) != 0 ? 1u : 0u);
      }
      umma_commit(&empty[s]);  // the slot is free once these instructions have read it
    }
    if (ok) {
      umma_commit(accum);  // the accumulator is complete once everything issued has finished
      committed = true;
    } else {
      atomicExch(p.status, (int)B2_ERR_TIMEOUT);
    }
  }
  __syncwarp();

  // ---- epilogue: every warp reads its 32 accumulator rows, 16 columns at a time
  bool done = true;
  if (KT > 0) {
    // Warp-uniform verdict: the accumulator load below is a warp-wide instruction.  Most threads start this wait
    // at kernel entry, so its limit grows with the length of the k-loop it has to outlast (a slab of this tile
    // takes well under a microsecond of tensor-pipe time; four are allowed).
    const uint64_t accum_limit = kWaitLimitNs + (uint64_t)KT * 4096ull;
    done = __all_sync(0xffffffffu, mbar_wait_bounded(accum, 0, accum_limit) ? 1 : 0) != 0;
    tc_fence_after();
    if (done) {
      const int64_t row = m0 + warp * 32 + lane;
      const uint32_t taddr = tmem_d + ((uint32_t)(warp * 32) << 16);
      const bool use_beta = (p.beta != 0.0f);
      // 32 columns per step: the old C values are requested first, so that their latency runs under the
      // accumulator load; both are complete before the first store.
      for (int c0 = 0; c0 < TBN; c0 += 32) {
        float old[32];
        if (use_beta && row < p.m) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int64_t col = n0 + c0 + j;
            old[j] = (col < p.n) ? p.C[row + col * p.ldc] : 0.0f;
          }
        }
        uint32_t r0[16], r1[16];
        tmem_ld16_issue(taddr + (uint32_t)c0, r0);  // all lanes take part (the loads are warp-wide)
        tmem_ld16_issue(taddr + (uint32_t)c0 + 16u, r1);
        tmem_ld_wait(r0, r1);
        if (row < p.m) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int64_t col = n0 + c0 + j;
            if (col < p.n) {
              float out = p.alpha * __uint_as_float(j < 16 ? r0[j] : r1[j - 16]);
              if (use_beta) out += p.beta * old[j];
              p.C[row + col * p.ldc] = out;
            }
          }
        }
      }
    } else if (lane == 0) {
      atomicExch(p.status, (int)B2_ERR_TIMEOUT);
    }
  }

  // ---- common exit: free the tensor memory.  The barrier below is reached by the producer only after its copies
  // have landed (or their bounded waits ran out).  If the epilogue gave up although the issuing thread had
  // committed the accumulator, multiply-adds may still be running: that thread waits for them once more (bounded)
  // before the tensor memory they write is freed.
  if (warp == 1 && lane == 0 && !done && committed) (void)mbar_wait_bounded(accum, 0, kWaitLimitNs);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_d, TBN);
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn tf32_lookup_encode_fn() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return reinterpret_cast<EncodeFn>(ptr);
  return nullptr;
}
EncodeFn tf32_encode_fn() {
  static const EncodeFn fn = tf32_lookup_encode_fn();  // initialised once, thread-safe
  return fn;
}

// Panel P[rows][pitch] (pitch floats, k contiguous): boxes of 32 k by box_rows rows, 128-byte swizzle.
bool panel_map(CUtensorMap* map, const float* P, int64_t rows, int64_t pitch, int box_rows) {
  EncodeFn enc = tf32_encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)pitch, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)TBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(P), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool t_is_n(char c) { return c == 'N' || c == 'n'; }

template <int TBN, int TSTAGES, int MINB = 1>
int launch_tf32(const Tf32Args& a, const float* PA, const float* PB, int64_t pitch, int dev, cudaStream_t st) {
  static std::atomic<bool> configured[64];
  auto kfn = sgemm_tf32_kernel<TBN, TSTAGES, MINB>;
  constexpr size_t smem = Tf32Cfg<TBN, TSTAGES>::SMEM_BYTES;
  if (!configured[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return B2_ERR_LAUNCH;
    configured[dev].store(true, std::memory_order_release);
  }
  CUtensorMap mapA, mapB;
  if (!panel_map(&mapA, PA, a.m, pitch, TBM) || !panel_map(&mapB, PB, a.n, pitch, TBN)) return B2_ERR_LAUNCH;
  const long long tiles = (long long)a.tiles_m * ((a.n + TBN - 1) / TBN);
  if (tiles > 0x7fffffffLL) return B2_ERR_LAUNCH;
  kfn<<<(unsigned)tiles, 128, smem, st>>>(a, mapA, mapB);
  return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
}

struct PackPlan {
  int64_t kpad, pitch;
  size_t off_b, total;
};
PackPlan pack_plan(int terms, int64_t m, int64_t n, int64_t k) {
  PackPlan p;
  p.kpad = (k + TBK - 1) / TBK * TBK;
  p.pitch = (int64_t)terms * p.kpad;
  const size_t sa = round_up((size_t)(m > 0 ? m : 0) * p.pitch * 4, 1024);
  const size_t sb = round_up((size_t)(n > 0 ? n : 0) * p.pitch * 4, 1024);
  p.off_b = sa, p.total = sa + sb;
  return p;
}

int sgemm_tf32(int terms, char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
               int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc, void* ws, size_t ws_bytes,
               void* cuda_stream) {
  const bool scale_only = (alpha == 0.0f || k == 0);
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  if (m == 0 || n == 0) return B2_OK;
  if (scale_only)  // C := beta*C needs no tensor cores
    return gemm_entry<float>(B2_VARIANT_AUTO, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cuda_stream);
  // 32-bit tile coordinates; the pack kernel walks the rows of an operand in 64-row blocks of the grid's second
  // dimension (at most 65535 blocks)
  constexpr int64_t kMaxRows = 65535LL * 64;
  if (m > kMaxRows || n > kMaxRows || k > 0x2aaaaaaaLL) return B2_ERR_VARIANT;
  const PackPlan pl = pack_plan(terms, m, n, k);
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < pl.total) return B2_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  float* PA = reinterpret_cast<float*>(ws);
  float* PB = reinterpret_cast<float*>(static_cast<char*>(ws) + pl.off_b);

  static std::atomic<int*> status_by_device[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return B2_ERR_LAUNCH;
  if (!status_by_device[dev].load(std::memory_order_acquire)) {
    void* sp = nullptr;
    if (cudaGetSymbolAddress(&sp, g_tf32_status) != cudaSuccess) return B2_ERR_LAUNCH;
    status_by_device[dev].store(static_cast<int*>(sp), std::memory_order_release);
  }

  // step 1: pack.  op(A)(i, p): A[i + p*lda] (N) or A[p + i*lda] (T);  op(B)^T(j, p): B[p + j*ldb] (N) or B[j + p*ldb] (T)
  const dim3 pb(256);
  const dim3 ga((unsigned)((pl.kpad + 63) / 64), (unsigned)((m + 63) / 64)), gb((unsigned)((pl.kpad + 63) / 64), (unsigned)((n + 63) / 64));
  if (t_is_n(transa))
    tf32_pack_kernel<false><<<ga, pb, 0, st>>>(A, lda, m, k, pl.kpad, terms, true, PA);
  else
    tf32_pack_kernel<true><<<ga, pb, 0, st>>>(A, lda, m, k, pl.kpad, terms, true, PA);
  if (t_is_n(transb))
    tf32_pack_kernel<true><<<gb, pb, 0, st>>>(B, ldb, n, k, pl.kpad, terms, false, PB);
  else
    tf32_pack_kernel<false><<<gb, pb, 0, st>>>(B, ldb, n, k, pl.kpad, terms, false, PB);
  if (cudaGetLastError() != cudaSuccess) return B2_ERR_LAUNCH;

  // step 2: multiply
  Tf32Args a;
  a.m = m, a.n = n, a.kt = (int)(pl.pitch / TBK), a.alpha = alpha, a.beta = beta, a.C = C, a.ldc = ldc;
  a.tiles_m = (int)((m + TBM - 1) / TBM);
  a.status = status_by_device[dev];
  // wide tiles unless they would leave SMs without work that narrow tiles can fill
  const long long wide_tiles = (long long)a.tiles_m * ((n + 255) / 256);
  if (n > 128 && wide_tiles >= 96) {
    // More than one wave of tiles and a main loop short enough for the epilogue to matter: two CTAs per SM, each
    // with a 2-stage ring (96 KB) and 256 of the 512 tensor-memory columns, so that one CTA's epilogue and ramp-up
    // run under the other's multiply-adds.  Measured (TFLOP/s, packing included, against one CTA with 4 stages):
    // 3072^3 440 / 386, 4096^3 476 / 412, 8192^3 663 / 592, three-term 4096^3 200 / 187, 8192^3 225 / 228.
    if (wide_tiles > sm_count_cached() && a.kt <= 512) return launch_tf32<256, 2, 2>(a, PA, PB, pl.pitch, dev, st);
    return launch_tf32<256, 4>(a, PA, PB, pl.pitch, dev, st);
  }
  return launch_tf32<128, 6>(a, PA, PB, pl.pitch, dev, st);
}

}  // namespace

// status word of the TF32 kernels, merged into b2_device_status by gemm_f64_tma.cu
int tf32_take_status() {
  int value = 0;
  if (cudaMemcpyFromSymbol(&value, g_tf32_status, sizeof(int)) != cudaSuccess) return B2_ERR_LAUNCH;
  if (value != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_tf32_status, &zero, sizeof(int)) != cudaSuccess) return B2_ERR_LAUNCH;
  }
  return value;
}

}  // namespace b2

extern "C" size_t b2_sgemm_tf32_workspace_bytes(int terms, int64_t m, int64_t n, int64_t k) {
  if ((terms != 1 && terms != 3) || m < 0 || n < 0 || k < 0) return 0;
  return b2::pack_plan(terms, m, n, k).total;
}

extern "C" int b2_sgemm_tf32x1(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                               int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::sgemm_tf32(1, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, workspace_bytes,
                        cuda_stream);
}

extern "C" int b2_sgemm_tf32x3(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                               int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return b2::sgemm_tf32(3, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, workspace_bytes,
                        cuda_stream);
}
