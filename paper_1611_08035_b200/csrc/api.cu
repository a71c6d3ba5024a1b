// C-ABI entry points of the real GEMM: argument checking, quick returns, variant selection.
#include <cuda_runtime.h>

#include <atomic>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "b2gemm.h"
#include "entry.h"
#include "gemm_launch.cuh"
#include "queue_model.h"
#include "select.h"

namespace b2 {

int launch_f64_v0(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v1(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v2(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v3(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v4(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v5(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_v6(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_t32(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_tma_t32(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_w8(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_ws_64x64(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f64_ws_64x64_direct(const GemmArgs<double>&, bool, bool, bool, cudaStream_t);
int launch_f32_v0(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);
int launch_f32_v1(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);
int launch_f32_v2(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);
int launch_f32_v3(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);
int launch_f32_s32(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);
int launch_f32_tma(const GemmArgs<float>&, bool, bool, bool, cudaStream_t);

model::SmPrediction predict_variant(int dtype, int variant);  // model_api.cu

namespace {

constexpr double kModelTrust = 0.04;

// name, micro-kernel, BM, BN, BK, stages, threads, resident CTAs per SM, measured steady-state efficiency
const VariantInfo kF64Info[] = {
    {"dmma_128x128x16_s4", "dmma", 128, 128, 16, 4, 256, 1, 0.87},
    {"dmma_128x64x16_s3", "dmma", 128, 64, 16, 3, 128, 2, 0.94},
    {"dmma_64x64x16_s3", "dmma", 64, 64, 16, 3, 128, 4, 0.955},
    {"dfma_128x64x16_s3", "dfma", 128, 64, 16, 3, 128, 2, 0.73},
    {"dmma_tma_64x64x16_s3", "dmma_tma", 64, 64, 16, 3, 128, 4, 0.97},
    {"dmma_tma_128x64x16_s3", "dmma_tma", 128, 64, 16, 3, 128, 2, 0.945},
    {"dmma_tma_128x128x16_s4", "dmma_tma", 128, 128, 16, 4, 256, 1, 0.95},
    {"dmma_32x32x16_s3", "dmma", 32, 32, 16, 3, 128, 7, 0.80, 8, 8, 0.0, 7.0, true},
    {"dmma_tma_32x32x16_s3", "dmma_tma", 32, 32, 16, 3, 128, 6, 0.80},
    {"dmma_w8_64x64x16_s3", "dmma_w8", 64, 64, 16, 3, 256, 3, 0.91},
    {"dmma_ws_3x64x64x16_s3", "dmma_ws", 64, 64, 16, 3, 512, 1, 0.95},
    {"dmma_ws_direct_3x64x64x16_s3", "dmma_ws", 64, 64, 16, 3, 512, 1, 0.95},
};
const LaunchFn<double> kF64Launch[] = {launch_f64_v0, launch_f64_v1, launch_f64_v2, launch_f64_v3,
                                       launch_f64_v4, launch_f64_v5, launch_f64_v6, launch_f64_t32,
                                       launch_f64_tma_t32, launch_f64_w8, launch_f64_ws_64x64,
                                       launch_f64_ws_64x64_direct};
const VariantInfo kF32Info[] = {
    {"ffma2_t16x8_128x128x16_s3", "ffma2", 128, 128, 16, 3, 128, 2, 0.782, 16, 8, 3500.0, 11.0},
    {"ffma2_128x64x16_s4", "ffma2", 128, 64, 16, 4, 128, 3, 0.795, 8, 8, 0.0, 5.8, true},
    {"ffma2_64x64x16_s4", "ffma2", 64, 64, 16, 4, 64, 6, 0.64},
    {"ffma_128x64x16_s4", "ffma", 128, 64, 16, 4, 128, 4, 0.70},
    {"ffma2_t4_32x32x16_s4", "ffma2", 32, 32, 16, 4, 64, 8, 0.40, 4, 4, 0.0, 7.0, true},
    {"ffma2_tma_128x128x16_s6", "ffma2_tma", 128, 128, 16, 6, 128, 2, 0.785, 16, 8, 3500.0},
};
const LaunchFn<float> kF32Launch[] = {launch_f32_v0, launch_f32_v1, launch_f32_v2,
                                      launch_f32_v3, launch_f32_s32, launch_f32_tma};

}  // namespace

int f64_variant_count() { return (int)(sizeof(kF64Info) / sizeof(kF64Info[0])); }
const VariantInfo& f64_variant_info(int v) { return kF64Info[v]; }
LaunchFn<double> f64_variant_launch(int v) { return kF64Launch[v]; }
int f32_variant_count() { return (int)(sizeof(kF32Info) / sizeof(kF32Info[0])); }
const VariantInfo& f32_variant_info(int v) { return kF32Info[v]; }
LaunchFn<float> f32_variant_launch(int v) { return kF32Launch[v]; }

static bool is_n(char c) { return c == 'N' || c == 'n'; }
static bool is_t(char c) { return c == 'T' || c == 't' || c == 'C' || c == 'c'; }

// BLAS argument check; 0 or the negative index of the first illegal argument.
int check_gemm_args(char transa, char transb, int64_t m, int64_t n, int64_t k, const void* A, int64_t lda,
                    const void* B, int64_t ldb, const void* C, int64_t ldc, bool reads_ab) {
  if (!is_n(transa) && !is_t(transa)) return -1;
  if (!is_n(transb) && !is_t(transb)) return -2;
  if (m < 0) return -3;
  if (n < 0) return -4;
  if (k < 0) return -5;
  const int64_t rows_a = is_n(transa) ? m : k, rows_b = is_n(transb) ? k : n;
  const bool nonempty = m > 0 && n > 0;
  if (nonempty && reads_ab && !A) return -7;
  if (lda < (rows_a > 1 ? rows_a : 1)) return -8;
  if (nonempty && reads_ab && !B) return -9;
  if (ldb < (rows_b > 1 ? rows_b : 1)) return -10;
  if (nonempty && !C) return -12;
  if (ldc < (m > 1 ? m : 1)) return -13;
  return 0;
}

int sm_count_cached() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int sms = cached[dev].load(std::memory_order_relaxed);
  if (sms == 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    cached[dev].store(sms, std::memory_order_relaxed);
  }
  return sms;
}

template <typename T>
static int variant_count_t();
template <>
int variant_count_t<double>() { return f64_variant_count(); }
template <>
int variant_count_t<float>() { return f32_variant_count(); }
template <typename T>
static const VariantInfo& variant_info_t(int v);
template <>
const VariantInfo& variant_info_t<double>(int v) { return f64_variant_info(v); }
template <>
const VariantInfo& variant_info_t<float>(int v) { return f32_variant_info(v); }
template <typename T>
static LaunchFn<T> variant_launch_t(int v);
template <>
LaunchFn<double> variant_launch_t<double>(int v) { return f64_variant_launch(v); }
template <>
LaunchFn<float> variant_launch_t<float>(int v) { return f32_variant_launch(v); }

template <typename T>
static bool operands_aligned(const T* A, int64_t lda, const T* B, int64_t ldb) {
  constexpr int VEC = 16 / (int)sizeof(T);
  return ((reinterpret_cast<uintptr_t>(A) & 15) == 0) && ((reinterpret_cast<uintptr_t>(B) & 15) == 0) &&
         (lda % VEC == 0) && (ldb % VEC == 0);
}

// `aligned`: A and B have 16-byte aligned columns (16-byte staging); the TMA-staged variants need that and a
// single problem (`batch` <= 1).
// ta / tb: op(A) = A^T, op(B) = B^T.  They matter to the FMA micro-kernels only, which want both operands packed
// with the C index contiguous and copy a k-contiguous operand (A when ta, B when not tb) element by element.
// ksplit_out (optional): where a variant can split the k-loop of a tile over a cluster of 2 or 4 CTAs, the same
// estimate is made for the problem seen as 2 or 4 times the tiles with a half or a quarter of k, plus what the
// reduction costs a tile; the best (variant, split) pair wins.  Measured with the 128 x 64 fp32 tile (us, split 1 /
// 2 / 4): 768^3 45.1 / 28.7 / 36.9, 1024^3 57.9 / 53.7 / 58.0, 1536^3 141 / 142 / 162, 2048^3 355 / 312 / 343,
// 3072^3 1031 / 1031 / 1086.
template <typename T>
int choose_variant_uncached(int64_t m, int64_t n, int64_t k, bool aligned, int64_t batch, bool ta, bool tb,
                            int* ksplit_out, bool drain_free);

// The choice is a pure function of its arguments (and of the device's SM count) that costs a few microseconds of
// model arithmetic: as much as a small problem's kernel.  Each host thread remembers its last few choices.
template <typename T>
int choose_variant(int64_t m, int64_t n, int64_t k, bool aligned, int64_t batch = 1, bool ta = false,
                   bool tb = false, int* ksplit_out = nullptr, bool drain_free = false) {
  struct Entry {
    int64_t m, n, k, batch;
    int flags, sms, variant, ksplit;
  };
  constexpr int kEntries = 16;
  thread_local Entry cache[kEntries] = {};
  thread_local int next = 0;
  const int flags = 1 | (aligned ? 2 : 0) | (ta ? 4 : 0) | (tb ? 8 : 0) | (ksplit_out ? 16 : 0) |
                    (drain_free ? 32 : 0);  // never 0
  const int sms = sm_count_cached();
  for (int i = 0; i < kEntries; ++i) {
    const Entry& e = cache[i];
    if (e.flags == flags && e.m == m && e.n == n && e.k == k && e.batch == batch && e.sms == sms) {
      if (ksplit_out) *ksplit_out = e.ksplit;
      return e.variant;
    }
  }
  int ksplit = 1;
  const int v = choose_variant_uncached<T>(m, n, k, aligned, batch, ta, tb, ksplit_out ? &ksplit : nullptr, drain_free);
  cache[next] = Entry{m, n, k, batch, flags, sms, v, ksplit};
  next = (next + 1) % kEntries;
  if (ksplit_out) *ksplit_out = ksplit;
  return v;
}

template <typename T>
int choose_variant_uncached(int64_t m, int64_t n, int64_t k, bool aligned, int64_t batch, bool ta, bool tb,
                            int* ksplit_out, bool drain_free) {
  // tensor-map coordinates are 32-bit
  const bool tma_ok = aligned && batch <= 1 && m <= 0x7fffffffLL && n <= 0x7fffffffLL && k <= 0x7fffffffLL;
  const int count = variant_count_t<T>();
  TileChoice cand[16];
  for (int v = 0; v < count && v < 16; ++v) {
    const VariantInfo& vi = variant_info_t<T>(v);
    // measured counterparts, never chosen automatically: the FMA micro-kernels on fp64 / scalar fp32, the
    // eight-warp 64 x 64 tile (slower than the four-warp one wherever it was measured) and the persistent kernel
    const bool comparison_only = strcmp(vi.micro, "dfma") == 0 || strcmp(vi.micro, "ffma") == 0 ||
                                 strcmp(vi.micro, "dmma_ws") == 0 || strcmp(vi.micro, "dmma_w8") == 0;
    // the TMA-staged fp32 kernel wins only where both operands have their C index contiguous (A not transposed, B
    // transposed: no transposition anywhere), and serves plain single problems only (ksplit_out is null for
    // triangular updates)
    const bool fp32_tma = strcmp(vi.micro, "ffma2_tma") == 0;
    // ... and, for updates of up to 1024 in k whose tiles leave through shared memory (drain_free: beta is 0 or 1
    // and the columns of C are 16-byte aligned), in NN and TT as well: measured at 2048^2 to 16384^2 with k = 64 to
    // 2048, e.g. 16384^2 x 64, beta = 1: 51.0 against 43.1 TFLOP/s, x 256: 57.5 against 54.8, x 1024: 59.2 against 58.8
    const bool short_update = drain_free && k <= 1024 && !(ta && !tb);
    const bool fp32_tma_fits = ((!ta && tb) || short_update) && ksplit_out != nullptr;
    const bool needs_alignment = strcmp(vi.micro, "dmma_tma") == 0 || strcmp(vi.micro, "ffma2_tma") == 0;
    // Steady-state fraction of the arithmetic pipe at full residency: the pipeline model's prediction (Section 4
    // estimate x latency coverage x barrier stall, queue_model.h).  The table's measured value is the recorded check
    // of that prediction; it replaces it only where the two are more than kModelTrust apart (fp32 tiles whose
    // element-wise transposing copies the model does not price, the 32 x 32 cp.async tile).
    const model::SmPrediction pr = predict_variant(sizeof(T) == 8 ? B2_F64 : B2_F32, v);
    double eff = (pr.feasible && fabs(pr.fraction - vi.efficiency) <= kModelTrust) ? pr.fraction : vi.efficiency;
    // Unaligned operands are staged in 8- or 4-byte pieces: twice to four times the staging instructions, which
    // weigh the more the smaller the tile (staging work per multiply-add goes with (BM+BN)/(BM*BN)); measured on
    // the 1001 x 999 x 1003 problem with odd leading dimensions.
    if (!aligned) eff *= 1.0 - 3.2 * (double)(vi.bm + vi.bn) / ((double)vi.bm * vi.bn);
    // Element-wise transposing copies (FMA micro-kernels): the table's efficiency is measured in NN, where B is
    // copied that way; the loss goes with the copied elements per multiply-add, 1/BN for A and 1/BM for B.
    // Measured at 8192^3 (128 x 64 tile, TFLOP/s): NT 62.0, NN 59.2, TT 51.3, TN 47.1; 128 x 128: 63.7, 58.2, 56.8, 54.9.
    // The cost of B's copy differs per variant (128 x 64 transposes it through registers).
    if (fp32_tma) {
      eff = (!ta && tb) ? 0.868 : 0.86;  // NT at 8192^3; the short updates are set above the cp.async kernels
    } else if (strncmp(vi.micro, "ffma", 4) == 0 && sizeof(T) == 4) {
      const double ca = 10.0, cb = vi.transpose_b_cost;  // fitted to the eight figures above (within 4 %)
      double f = (1.0 - (ta ? ca / vi.bn : 0.0) - (tb ? 0.0 : cb / vi.bm)) / (1.0 - cb / vi.bm);
      if (f > 1.15) f = 1.15;  // the 32 x 32 tile gains 1.24-1.32 in NT, but the estimate already favours it at 1024^3
      eff *= f;
    }
    cand[v] = TileChoice{vi.bm, vi.bn, vi.bk, vi.threads, vi.ctas_per_sm, eff,
                         comparison_only || (needs_alignment && !tma_ok) || (fp32_tma && !fp32_tma_fits)};
    // measured: a TMA-staged CTA starts about 2 microseconds later than a cp.async one (512^3: 17.4 against 12.6 us)
    if (needs_alignment) cand[v].extra_fixed_clks = 4500.0;
    cand[v].per_tile_extra_clks = vi.per_tile_extra_clks;
  }
  const int sms = sm_count_cached();
  int best = select_tile(cand, count < 16 ? count : 16, m, n, k, sms, (int)sizeof(T), batch);
  // fp32 updates of up to 1024 in k whose tiles leave through shared memory, at least one and a half tiles of
  // 128 x 128 per SM: the TMA-staged kernel is the measured best by 5 to 20 % in NN, NT and TT, which the estimate,
  // fitted to kernels with the ordinary epilogue, does not see (2048^2 x 128: 35.5 against 31.6 TFLOP/s; below
  // that tile count it loses: 1024^2 x 256 16.7 against 24.5)
  if (sizeof(T) == 4 && drain_free && k <= 1024 && !(ta && !tb) && tma_ok && batch <= 1 && ksplit_out != nullptr) {
    for (int v = 0; v < count && v < 16; ++v) {
      const VariantInfo& vi = variant_info_t<T>(v);
      if (strcmp(vi.micro, "ffma2_tma") != 0) continue;
      const int64_t tiles = ((m + vi.bm - 1) / vi.bm) * ((n + vi.bn - 1) / vi.bn);
      if (2 * tiles >= 3 * (int64_t)sms) {
        *ksplit_out = 1;
        return v;
      }
    }
  }
  if (ksplit_out) {
    *ksplit_out = 1;
    double best_t = estimate_clks(cand[best], m, n, k, sms, (int)sizeof(T), batch);
    for (int v = 0; v < count && v < 16; ++v) {
      const VariantInfo& vi = variant_info_t<T>(v);
      if (!vi.can_ksplit || cand[v].explicit_only) continue;
      for (int split = 2; split <= 2; split *= 2) {  // 4 CTAs per tile never beat the better of 1 and 2 where measured
        const int64_t slabs = (k + vi.bk - 1) / vi.bk;
        if (slabs < 8 * split) break;  // keep at least 8 slabs per CTA
        // with fewer tiles than a quarter of the SMs the 32 x 32 tile is the better tool (512^3 TN: 18.5 us against 24.4)
        const int64_t tiles = ((m + vi.bm - 1) / vi.bm) * ((n + vi.bn - 1) / vi.bn) * (batch < 1 ? 1 : batch);
        if (4 * tiles < sms) break;
        // small tiles that fill an SM with six or more CTAs gain from a split only while the tiles themselves are
        // fewer than about one per SM (measured: 32 x 32 tiles, both data types, split better at 256^3 and 384^3,
        // 64 and 144 tiles, worse at 512^3, 256 tiles)
        if (vi.ctas_per_sm >= 6 && 4 * tiles > 5 * (int64_t)sms) break;
        const int64_t k_part = (slabs + split - 1) / split * vi.bk;
        TileChoice c = cand[v];
        // reduction: two cluster barriers and, for the first CTA, the other CTAs' accumulators through
        // distributed shared memory
        // (about 2000 clocks for the 128 x 64 fp32 tile, where it was fitted; 800 for a 32 x 32 fp64 tile)
        c.per_tile_extra_clks += 400.0 + (split - 1) * (double)vi.bm * vi.bn * sizeof(T) / 10.0 / split;
        const double t = estimate_clks(c, m, n, k_part, sms, (int)sizeof(T), batch * split);
        if (t < 0.97 * best_t) best = v, best_t = t, *ksplit_out = split;  // a split has to win by 3 %
      }
    }
  }
  return best;
}

// Variant choice and launch of an already checked, non-trivial problem (m, n, k > 0, alpha != 0).
template <typename T>
int gemm_launch_checked(int variant, bool ta, bool tb, int64_t m, int64_t n, int64_t k, T alpha, const T* A,
                        int64_t lda, const T* B, int64_t ldb, T beta, T* C, int64_t ldc, const GemmExtra& ex,
                        cudaStream_t stream) {
  // TMA staging needs 16-byte aligned columns and one tensor map per operand, so it serves single problems only
  // (every problem of a batch must start on a 16-byte boundary for the 16-byte staging path)
  constexpr int64_t kVec = 16 / (int64_t)sizeof(T);
  const bool aligned = operands_aligned(A, lda, B, ldb) &&
                       (ex.batch <= 1 || (ex.stride_a % kVec == 0 && ex.stride_b % kVec == 0));
  int ksplit = ex.ksplit > 0 ? ex.ksplit : 1;
  if (variant == B2_VARIANT_AUTO)
    variant = choose_variant<T>(m, n, k, aligned, ex.batch, ta, tb, ex.tri == 0 ? &ksplit : nullptr,
                                (beta == T(0) || beta == T(1)) && (reinterpret_cast<uintptr_t>(C) & 15) == 0 &&
                                    ldc % kVec == 0);
  GemmArgs<T> args;
  args.m = m, args.n = n, args.k = k;
  args.alpha = alpha, args.beta = beta;
  args.A = A, args.lda = lda, args.B = B, args.ldb = ldb, args.C = C, args.ldc = ldc;
  args.tiles_m = args.tiles_n = 0;
  args.ksplit = ksplit;
  args.tri = ex.tri;
  args.batch = ex.batch, args.batch_a = ex.stride_a, args.batch_b = ex.stride_b, args.batch_c = ex.stride_c;
  // Rasterisation group: the CTAs resident at one time should cover a block of C whose A row-panels and
  // B column-panels have about the same size: group_m * BM = (resident / group_m) * BN.
  const VariantInfo& vi = variant_info_t<T>(variant);
  const double resident = (double)sm_count_cached() * vi.ctas_per_sm;
  int group_m = (int)(sqrt(resident * vi.bn / vi.bm) + 0.5);
  // Measured at 8192^3 (DRAM bytes of one launch): 12 tile rows per group read the least for every tile shape
  // (64x64: 13.2 GB against 15.8 GB at 24 rows and 64 GB without grouping; 128x128: 7.6 GB), at unchanged speed.
  if (group_m > 12) group_m = 12;
  args.group_m = group_m < 1 ? 1 : group_m;
  return variant_launch_t<T>(variant)(args, ta, tb, aligned, stream);
}
template int gemm_launch_checked<double>(int, bool, bool, int64_t, int64_t, int64_t, double, const double*, int64_t,
                                         const double*, int64_t, double, double*, int64_t, const GemmExtra&,
                                         cudaStream_t);
template int gemm_launch_checked<float>(int, bool, bool, int64_t, int64_t, int64_t, float, const float*, int64_t,
                                        const float*, int64_t, float, float*, int64_t, const GemmExtra&, cudaStream_t);

template <typename T>
int gemm_entry(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, T alpha, const T* A,
               int64_t lda, const T* B, int64_t ldb, T beta, T* C, int64_t ldc, void* cuda_stream) {
  const bool scale_only = (alpha == T(0) || k == 0);
  const int bad = check_gemm_args(transa, transb, m, n, k, A, lda, B, ldb, C, ldc, !scale_only);
  if (bad) return bad;
  // an explicit variant may carry a k split request: variant + 256 * (CTAs per tile)
  GemmExtra ex;
  if (variant >= 256) {
    ex.ksplit = variant >> 8;
    variant &= 255;
    if (ex.ksplit != 2 && ex.ksplit != 4) return B2_ERR_VARIANT;
  }
  if (variant != B2_VARIANT_AUTO && (variant < 0 || variant >= variant_count_t<T>())) return B2_ERR_VARIANT;
  if (m == 0 || n == 0) return B2_OK;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (scale_only) {
    if (beta == T(1)) return B2_OK;
    const int64_t total = m * n;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count_cached() * 16;
    if (blocks > cap) blocks = cap;
    scale_kernel<T><<<(unsigned)blocks, threads, 0, stream>>>(m, n, beta, C, ldc);
    return cudaGetLastError() == cudaSuccess ? B2_OK : B2_ERR_LAUNCH;
  }
  return gemm_launch_checked<T>(variant, is_t(transa), is_t(transb), m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                                ex, stream);
}

// Explicit instantiations used by the other translation units (complex and host-buffer entries).
template int gemm_entry<double>(int, char, char, int64_t, int64_t, int64_t, double, const double*, int64_t,
                                const double*, int64_t, double, double*, int64_t, void*);
template int gemm_entry<float>(int, char, char, int64_t, int64_t, int64_t, float, const float*, int64_t, const float*,
                               int64_t, float, float*, int64_t, void*);

}  // namespace b2

extern "C" int b2_dgemm(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                        int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                        void* cuda_stream) {
  return b2::gemm_entry<double>(B2_VARIANT_AUTO, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                                cuda_stream);
}

extern "C" int b2_sgemm(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                        int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                        void* cuda_stream) {
  return b2::gemm_entry<float>(B2_VARIANT_AUTO, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                               cuda_stream);
}

extern "C" int b2_dgemm_variant(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha,
                                const double* A, int64_t lda, const double* B, int64_t ldb, double beta, double* C,
                                int64_t ldc, void* cuda_stream) {
  return b2::gemm_entry<double>(variant, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cuda_stream);
}

extern "C" int b2_sgemm_variant(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha,
                                const float* A, int64_t lda, const float* B, int64_t ldb, float beta, float* C,
                                int64_t ldc, void* cuda_stream) {
  return b2::gemm_entry<float>(variant, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, cuda_stream);
}

extern "C" int b2_variant_count(int dtype) {
  if (dtype == B2_F64) return b2::f64_variant_count();
  if (dtype == B2_F32) return b2::f32_variant_count();
  return 0;
}

extern "C" const char* b2_variant_name(int dtype, int variant) {
  if (variant < 0 || variant >= b2_variant_count(dtype)) return nullptr;
  return dtype == B2_F64 ? b2::f64_variant_info(variant).name : b2::f32_variant_info(variant).name;
}

extern "C" int b2_gemm_query_config(int dtype, char transa, char transb, int64_t m, int64_t n, int64_t k, int64_t lda,
                                    int64_t ldb, int64_t ldc, char* json_out, size_t cap) {
  if (dtype != B2_F64 && dtype != B2_F32) return -1;
  // dummy non-null pointers: only sizes and leading dimensions are checked here
  const void* dummy = reinterpret_cast<const void*>(16);
  const int bad = b2::check_gemm_args(transa, transb, m, n, k, dummy, lda, dummy, ldb, dummy, ldc, true);
  if (bad) return bad - 1;
  if (!json_out) return -11;
  const int elem = dtype == B2_F64 ? 8 : 4;
  const bool ld_aligned = (lda % (16 / elem) == 0) && (ldb % (16 / elem) == 0);
  const bool ta = b2::is_t(transa), tb = b2::is_t(transb);
  int ksplit = 1;
  const int v = dtype == B2_F64 ? b2::choose_variant<double>(m, n, k, ld_aligned, 1, ta, tb, &ksplit)
                                : b2::choose_variant<float>(m, n, k, ld_aligned, 1, ta, tb, &ksplit);
  const b2::VariantInfo& vi = dtype == B2_F64 ? b2::f64_variant_info(v) : b2::f32_variant_info(v);
  const long long tiles_m = (m + vi.bm - 1) / vi.bm, tiles_n = (n + vi.bn - 1) / vi.bn;
  char buf[768];
  const int len = snprintf(
      buf, sizeof(buf),
      "{\"dtype\": \"%s\", \"variant\": %d, \"name\": \"%s\", \"micro_kernel\": \"%s\", \"BM\": %d, \"BN\": %d, "
      "\"kc\": %d, \"stages\": %d, \"threads\": %d, \"ctas_per_sm\": %d, \"grid\": %lld, \"tiles_m\": %lld, "
      "\"tiles_n\": %lld, \"k_slabs\": %lld, \"k_split\": %d, \"vector_staging_if_pointers_aligned\": %s, \"sm_count\": %d}",
      dtype == B2_F64 ? "f64" : "f32", v, vi.name, vi.micro, vi.bm, vi.bn, vi.bk, vi.stages, vi.threads,
      vi.ctas_per_sm, tiles_m * tiles_n * ksplit, tiles_m, tiles_n, (long long)((k + vi.bk - 1) / vi.bk), ksplit,
      ld_aligned ? "true" : "false", b2::sm_count_cached());
  if (len < 0 || (size_t)len + 1 > cap) return B2_ERR_WORKSPACE;
  memcpy(json_out, buf, (size_t)len + 1);
  return B2_OK;
}

extern "C" const char* b2_version(void) { return "b2gemm 0.1 (sm_100a)"; }

extern "C" const char* b2_strerror(int status) {
  switch (status) {
    case B2_OK: return "success";
    case B2_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case B2_ERR_LAUNCH: return "CUDA launch or copy failed";
    case B2_ERR_WORKSPACE: return "workspace or output buffer null, misaligned or too small";
    case B2_ERR_VARIANT: return "unknown or inapplicable kernel variant";
    case B2_ERR_STATIC_LIMIT: return "problem needs more scratch than the built-in array of b2_zgemm4m_static holds";
    case -1: return "argument 1 is illegal";
    case -2: return "argument 2 is illegal";
    case -3: return "argument 3 is illegal";
    case -4: return "argument 4 is illegal";
    case -5: return "argument 5 is illegal";
    case -6: return "argument 6 is illegal";
    case -7: return "argument 7 is illegal";
    case -8: return "argument 8 is illegal";
    case -9: return "argument 9 is illegal";
    case -10: return "argument 10 is illegal";
    case -11: return "argument 11 is illegal";
    case -12: return "argument 12 is illegal";
    case -13: return "argument 13 is illegal";
    case -14: return "argument 14 is illegal";
    default: return status < 0 ? "illegal argument" : "unknown status";
  }
}
