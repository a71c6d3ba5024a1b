// The paper's analytical model (host code, no CUDA): throughput of an instruction mix from
// per-pipeline rates (Section 4) and the register limit on unit updates (Section 5), plus the
// same estimate re-targeted at one SM sub-partition for the micro-kernels of this library.
#pragma once
#include <math.h>
#include <stdint.h>

namespace b2 {
namespace model {

// Section 4 ("Little's Law"): a machine is a set of pipelines (queues) with throughputs rate[i]
// instructions per cycle; an instruction mix puts jobs[i] instructions on pipeline i per outer
// product (an instruction that needs several units counts as a job on each).  The mix clears
// at the pace of its slowest pipeline: outer products per cycle = min_i rate[i] / jobs[i].
// Pipelines without jobs do not constrain the result.  Returns -1 for invalid input.
inline double throughput(int npipes, const double* rate, const double* jobs) {
  if (npipes <= 0 || !rate || !jobs) return -1.0;
  double best = INFINITY;
  for (int i = 0; i < npipes; ++i) {
    if (!(rate[i] > 0.0) || jobs[i] < 0.0) return -1.0;
    if (jobs[i] > 0.0) {
      const double t = rate[i] / jobs[i];
      if (t < best) best = t;
    }
  }
  return best;
}

// Section 4 ("Estimating throughput"): when n of a pipeline's instructions depend on each
// other and have latency k, the latency cannot be hidden and the L jobs wait W = L + n*k
// cycles, so the pipeline finishes 1/W outer products per cycle.
inline double stalled_throughput(double jobs, int n_dependent, double latency) {
  if (!(jobs > 0.0) || n_dependent < 0 || latency < 0.0) return -1.0;
  return 1.0 / (jobs + n_dependent * latency);
}

// Section 5 ("Limits imposed by registers"): unit updates that fit beside the accumulators,
// N = floor((R_total - mr*nr/v - R_A) / R_R), R_R = 2 without fused multiply-add and 1 with.
// Returns -1 for invalid input (N itself may be 0 or negative when the tile does not fit).
inline int register_updates(int r_total, int mr, int nr, int v, int r_a, int r_r, bool* ok) {
  *ok = (r_total > 0 && mr > 0 && nr > 0 && v > 0 && r_a >= 0 && r_r > 0);
  if (!*ok) return 0;
  return (int)floor(((double)r_total - (double)mr * nr / v - r_a) / r_r);
}

// Section 5: a register sub-block ms x ns is admissible when ms*ns <= N_updates * v.
inline bool sub_block_fits(int ms, int ns, int n_updates, int v) { return ms * ns <= n_updates * v; }

// ---- the same estimate for one SM sub-partition (B200) ----------------------------------------
// Pipelines of a sub-partition and their rates in warp-instructions (or wavefronts) per clock:
//   issue      1      every instruction of the mix
//   fp64       1/2    a DFMA warp-instruction occupies the 16-lane FP64 pipe for two clocks
//   tensor64   1/32   one mma.sync m16n8k4 f64 = 512 multiply-adds at 16 per clock
//   fp32       1      a FFMA warp-instruction; the packed pair FFMA2 counts as two jobs
//   lsu        1/4    shared-memory wavefronts (128 bytes each), one per clock per SM
// (64 FP64 and 128 FP32 multiply-adds per clock per SM are the rates the probes measure.)
enum Pipe { ISSUE = 0, FP64 = 1, TENSOR64 = 2, FP32 = 3, LSU = 4, NPIPES = 5 };

inline void sm_rates(double (&rate)[NPIPES]) {
  rate[ISSUE] = 1.0, rate[FP64] = 0.5, rate[TENSOR64] = 1.0 / 32.0, rate[FP32] = 1.0, rate[LSU] = 0.25;
}

enum MicroKind { MK_DMMA = 0, MK_DFMA = 1, MK_FFMA = 2, MK_FFMA2 = 3 };

// Scalar 32-bit multiply-adds with three distinct register sources issue below one per clock when the compiler,
// not the programmer, places the operands (register-bank conflicts the packed 64-bit operands do not have); the
// same holds for FP64 multiply-adds on their pipe.  Slots per instruction, fitted to the two comparison kernels
// (scalar FFMA 0.70, DFMA 0.73 of peak); the tensor-core and packed-pair kernels carry no such factor.
constexpr double kScalarFmaSlots = 1.30;
constexpr double kDfmaSlots = 1.37;

// Jobs per pipeline for one rank-1 update (one k) of one warp's tile.
//   wtm x wtn     the warp's block of C (DMMA: 16x8 fragments; FMA kinds: 8 lanes x 4 lanes of tm x tn blocks,
//                 8 x 8 -> 64 x 32, 16 x 8 -> 128 x 32, 4 x 4 -> 32 x 16)
//   staging       cp.async instructions per thread per slab, slab_k = BK
struct WarpMix {
  double jobs[NPIPES];
  double fma_per_k;  // multiply-adds the warp performs per k
};

inline WarpMix warp_mix(int kind, int wtm, int wtn, int staging_per_slab, int slab_k) {
  WarpMix m;
  for (int i = 0; i < NPIPES; ++i) m.jobs[i] = 0.0;
  m.fma_per_k = (double)wtm * wtn;
  // staging (copy instruction plus its 64-bit address arithmetic), barrier, loop control per k: the profiler counts
  // 5.5 instructions per k beside the multiply-adds and fragment loads in the fp32 128 x 64 kernel, 7 to 8 in the
  // 128 x 128 one
  const double overhead = (staging_per_slab * 6.0 + 24.0) / slab_k;
  if (kind == MK_DMMA) {
    const double mi = wtm / 16.0, ni = wtn / 8.0;
    m.jobs[TENSOR64] = mi * ni / 4.0;           // one mma covers four k
    const double loads = (mi + ni) / 4.0;        // A: one 16-byte load per fragment row block, B: one 8-byte load
    m.jobs[LSU] = (mi * 4.0 + ni * 2.0) / 4.0;   // 512 and 256 distinct bytes per warp load
    m.jobs[ISSUE] = mi * ni / 4.0 + loads + overhead;
  } else {
    const double tm = wtm / 8.0, tn = wtn / 4.0;  // accumulator block per lane
    const double fma = tm * tn;
    const bool f64 = (kind == MK_DFMA);
    const double loads = (tm + tn) / (f64 ? 2.0 : 4.0);  // tm + tn operand values per lane in 16-byte loads
    m.jobs[LSU] = loads;                         // lanes of a warp share operands: one wavefront per load
    if (kind == MK_DFMA) {
      m.jobs[FP64] = fma * kDfmaSlots;
      m.jobs[ISSUE] = fma + loads + overhead;
    } else if (kind == MK_FFMA) {
      m.jobs[FP32] = fma;
      m.jobs[ISSUE] = fma * kScalarFmaSlots + loads + overhead;
    } else {
      // A packed pair instruction is two jobs on the FP32 pipe and holds the sub-partition's dispatch port for two
      // clocks (it reads three 64-bit operands per lane); so does a 16-byte shared-memory load.  At peak the pair
      // instructions alone fill the port, and every other instruction takes its slots from them: the loop of an
      // 8 x 8 block needs 64 + 8 slots per rank-1 update, of a 16 x 8 block 128 + 12.  The instruction-mix probes
      // (the inner loops over resident slabs, nothing else) measure 0.87 and 0.92 of the pipe's peak; the raw
      // pair instruction reaches 0.97.  (Copying a value of b into both halves of a pair costs nothing: the
      // profiler counts no instruction for it.)
      m.jobs[FP32] = fma;
      m.jobs[ISSUE] = fma + 2.0 * loads + overhead;
    }
  }
  return m;
}

// Predicted fraction of the arithmetic pipe's peak: (rank-1 updates per clock) x (multiply-adds per
// update) / (peak multiply-adds per clock per sub-partition).
inline double predicted_fraction(const WarpMix& m, bool fp64_data) {
  double rate[NPIPES];
  sm_rates(rate);
  const double lam = throughput(NPIPES, rate, m.jobs);
  const double peak = fp64_data ? 16.0 : 32.0;
  const double f = lam * m.fma_per_k / peak;
  return f > 1.0 ? 1.0 : f;
}

// ---- latency coverage (Section 4, "Dealing with dependencies across pipelines") ------------------------
// The paper sizes mr x nr so that the multiply-adds of one outer product are independent and cover the pipeline's
// latency; when they do not, the dependent instructions wait (W = L + n*k).  On an SM the instructions that can
// cover a pipeline's latency are the independent arithmetic instructions of ALL warps resident on a scheduler:
// I = warps per scheduler x independent instructions per unit update.  By Little's law the pipeline is kept full
// once I exceeds latency x rate; the smooth form 1 - exp(-I / I0) is fitted to one measured point of the tensor
// pipe (the TMA-staged 32 x 32 tile: six CTAs of four warps, two tensor instructions per warp and k-step, I = 12,
// 0.80 of peak -> I0 = 7.5) and used for every pipeline.
constexpr double kCoverageI0 = 7.5;
// The stall term itself (W = L + n*k): kernels staged with cp.async pass one CTA-wide barrier per slab, at which
// every warp of the CTA waits for the slowest and for the first fragments of the new slab: n = 1 dependent step
// of k = kBarrierStallClks per slab, which the other CTAs resident on the SM cover in proportion to their number
// (fitted to the one-CTA 128 x 128 DMMA kernel, 0.87 of peak; the FMA pipes, whose instructions return in a few
// clocks instead of the tensor pipe's tens, refill sooner: fitted to the scalar FFMA kernel).  Kernels fed through
// mbarriers by the tensor memory accelerator have no such step.
constexpr double kBarrierStallClksTensor = 250.0;
constexpr double kBarrierStallClksFma = 30.0;

inline double latency_coverage(double independent_in_flight) {
  return independent_in_flight <= 0.0 ? 0.0 : 1.0 - exp(-independent_in_flight / kCoverageI0);
}

// Limits of one SM that bound a candidate (queried from the device by the caller; B200 values as defaults).
struct SmLimits {
  int regs_per_sm = 65536;
  int max_regs_per_thread = 255;
  int smem_per_sm = 233472;  // bytes usable by CTAs
  int max_warps_per_sm = 64;
  int max_ctas_per_sm = 32;
  double l2_feed_bytes_per_clk = 32.0;  // sustainable L2 -> shared-memory feed per SM
};

// A candidate micro-kernel/tile: kind, the warp's block of C, the warp grid of a CTA, slab depth and ring stages.
struct SmCandidate {
  int kind;              // MicroKind
  int wtm, wtn;          // warp tile
  int warps_m, warps_n;  // warps of a CTA along m and n
  int bk, stages;
  bool tma;              // operand slabs arrive by the tensor memory accelerator through mbarriers (no CTA-wide barrier)
};

struct SmPrediction {
  bool feasible;        // fits registers and shared memory with at least two unit updates of fragments in flight
  int bm, bn, threads;
  int acc_regs, frag_regs, regs_per_thread;  // accumulators, fragments of one unit update, total (double-buffered)
  int n_updates;        // Section 5: floor((R_thread - accumulators - R_A) / R_R), unit updates of fragments that fit
  int smem_bytes;       // ring of `stages` slabs
  int ctas_per_sm;
  double pipe_fraction; // Section 4 estimate: min over pipelines, as a fraction of the arithmetic pipe's peak
  double feed_fraction; // what the L2 -> shared-memory feed allows for this tile's bytes per multiply-add
  double coverage;      // latency coverage at full residency
  double stall;         // L / (L + n*k): the barrier stall of cp.async-staged kernels (1 for TMA-staged ones)
  double fraction;      // product: the predicted fraction of peak
};

constexpr int kAddressRegs = 24;  // R_A: addresses, loop counters, barrier state

inline SmPrediction predict(const SmCandidate& c, const SmLimits& lim, int elem_bytes) {
  SmPrediction r = {};
  const int w = elem_bytes / 4;  // 32-bit registers per value
  r.bm = c.wtm * c.warps_m, r.bn = c.wtn * c.warps_n, r.threads = 32 * c.warps_m * c.warps_n;
  r.acc_regs = c.wtm * c.wtn * w / 32;
  double indep;  // independent arithmetic instructions of a warp per unit update
  if (c.kind == MK_DMMA) {
    const int mi = c.wtm / 16, ni = c.wtn / 8;
    r.frag_regs = (2 * mi + ni) * w;  // a0, a1 per row block, b0 per column block
    indep = mi * ni;
  } else {
    const int tm = c.wtm / 8, tn = c.wtn / 4;
    r.frag_regs = (tm + tn) * w;
    indep = (c.kind == MK_FFMA2) ? tm * tn / 2.0 : tm * tn;
  }
  // Section 5 restated for a thread: the register limit leaves room for N unit updates' worth of fragments;
  // software pipelining needs two (the next unit update's fragments are loaded while the current one is multiplied).
  r.n_updates = (lim.max_regs_per_thread - r.acc_regs - kAddressRegs) / (r.frag_regs > 0 ? r.frag_regs : 1);
  r.regs_per_thread = r.acc_regs + 2 * r.frag_regs + kAddressRegs;
  const int regs_alloc = (r.regs_per_thread + 7) / 8 * 8;
  // ring: BK x (BM + BN) values per slab plus a few values of padding per line
  r.smem_bytes = c.stages * c.bk * (r.bm + r.bn + 8) * elem_bytes;
  const int by_regs = lim.regs_per_sm / (r.threads * regs_alloc);
  const int by_smem = lim.smem_per_sm / (r.smem_bytes + 1024);
  const int by_warps = lim.max_warps_per_sm / (r.threads / 32);
  int ctas = by_regs < by_smem ? by_regs : by_smem;
  if (by_warps < ctas) ctas = by_warps;
  if (lim.max_ctas_per_sm < ctas) ctas = lim.max_ctas_per_sm;
  r.ctas_per_sm = ctas;
  r.feasible = r.n_updates >= 2 && ctas >= 1 && r.regs_per_thread <= lim.max_regs_per_thread && c.wtm > 0 && c.wtn > 0;
  if (!r.feasible) return r;
  const int staging = (r.bm + r.bn) * c.bk * elem_bytes / 16 / r.threads;
  // slabs that the tensor memory accelerator brings cost the multiplying warps no copy instructions
  const WarpMix mix = warp_mix(c.kind, c.wtm, c.wtn, c.tma ? 0 : (staging > 0 ? staging : 1), c.bk);
  r.pipe_fraction = predicted_fraction(mix, elem_bytes == 8);
  const double fma_per_clk = elem_bytes == 8 ? 64.0 : 128.0;
  const double bytes_per_fma = (double)(r.bm + r.bn) * elem_bytes / ((double)r.bm * r.bn);
  const double feed = lim.l2_feed_bytes_per_clk / (fma_per_clk * bytes_per_fma);
  r.feed_fraction = feed > 1.0 ? 1.0 : feed;
  const double warps_per_scheduler = ctas * (r.threads / 32) / 4.0;
  r.coverage = latency_coverage(warps_per_scheduler * indep);
  // clocks the slowest pipeline needs for one slab of one warp, at the SM's full rate for this warp's share
  double rate[NPIPES];
  sm_rates(rate);
  double slab_clks = 0.0;
  for (int i = 0; i < NPIPES; ++i) {
    const double t = mix.jobs[i] / rate[i] * c.bk;
    if (t > slab_clks) slab_clks = t;
  }
  const double k_stall = (c.kind == MK_DMMA ? kBarrierStallClksTensor : kBarrierStallClksFma) / ctas;
  r.stall = c.tma ? 1.0 : stalled_throughput(slab_clks, 1, k_stall) * slab_clks;  // L / (L + n*k)
  const double bound = r.pipe_fraction < r.feed_fraction ? r.pipe_fraction : r.feed_fraction;
  r.fraction = bound * r.coverage * r.stall;
  return r;
}

}  // namespace model
}  // namespace b2
