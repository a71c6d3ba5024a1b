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
  const double overhead = (staging_per_slab * 3.0 + 12.0) / slab_k;  // staging, barrier, loop control per k
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
      m.jobs[FP64] = fma;
      m.jobs[ISSUE] = fma + loads + overhead;
    } else if (kind == MK_FFMA) {
      m.jobs[FP32] = fma;
      m.jobs[ISSUE] = fma + loads + overhead;
    } else {
      m.jobs[FP32] = fma;                        // 32 packed instructions, two jobs each
      m.jobs[ISSUE] = fma / 2.0 + loads + tn + overhead;  // plus the moves that duplicate the tn values of b
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

}  // namespace model
}  // namespace b2
