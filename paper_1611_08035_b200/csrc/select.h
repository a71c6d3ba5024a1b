// Analytic choice of the CTA tile (host code, no CUDA).
//
// The paper picks a micro-kernel by estimating, per candidate, the time its instruction mix
// needs to clear the slowest pipeline (Section 4, "Little's Law": throughput = min over
// pipelines of rate / jobs) and keeps the best.  The same idea one level up: for each
// candidate CTA tile, estimate the clocks one SM needs for its share of the tiles from the
// three "pipelines" a tile occupies -- the arithmetic pipe, the L2->shared-memory feed and the
// C traffic of the epilogue -- and keep the candidate with the smallest estimate.
#pragma once
#include <math.h>
#include <stdint.h>

namespace b2 {

struct TileChoice {
  int bm, bn, bk;
  int threads;
  int ctas_per_sm;   // CTAs of this variant that fit on one SM
  double efficiency;  // measured steady-state fraction of the arithmetic pipe's peak
  bool explicit_only;  // never chosen automatically (comparison variants)
  double extra_fixed_clks = 0.0;  // start-up cost beyond the common one (TMA: descriptor fetch, barrier set-up)
  double per_tile_extra_clks = 0.0;  // exposed ramp-up/epilogue time per tile (variants with few, large CTAs per SM)
};

// Measured / derived machine rates per SM (B200): FP64 and FP32 multiply-adds per clock, the
// L2->SM feed and the SM's share of HBM bandwidth in bytes per clock, and fixed per-tile costs.
struct MachineRates {
  double fma_per_clk;        // 64 (fp64: DFMA and DMMA alike), 128 (fp32 FFMA)
  double l2_bytes_per_clk;   // sustainable L2 -> shared-memory feed per SM
  double hbm_bytes_per_clk;  // HBM bytes per clock per SM (6.5 TB/s / 148 SMs / 1.965 GHz)
  double tile_fixed_clks;    // launch + pipeline ramp-up + drain of one CTA
};

inline MachineRates machine_rates(int elem_bytes) {
  MachineRates r;
  r.fma_per_clk = elem_bytes == 8 ? 64.0 : 128.0;
  r.l2_bytes_per_clk = 32.0;
  r.hbm_bytes_per_clk = 22.0;
  r.tile_fixed_clks = 4000.0;
  return r;
}

// Estimated clocks for one SM to finish its share of the problem with tile `c`.
// `batch` independent problems of this shape share one launch (their tiles fill the SMs together).
inline double estimate_clks(const TileChoice& c, int64_t m, int64_t n, int64_t k, int sms, int elem_bytes,
                            int64_t batch = 1) {
  const MachineRates r = machine_rates(elem_bytes);
  const double tiles = (double)((m + c.bm - 1) / c.bm) * (double)((n + c.bn - 1) / c.bn) * (double)(batch < 1 ? 1 : batch);
  const double kt = (double)((k + c.bk - 1) / c.bk);
  // tiles are handed out CTA by CTA; an SM ends up with ceil(tiles / sms) of them
  const double per_sm = (double)(int64_t)((tiles + sms - 1) / sms);
  const double fma_tile = (double)c.bm * c.bn * c.bk * kt;
  // The SM's tiles run ctas_per_sm at a time; the last, partial group runs with fewer resident warps.
  const double cps = (double)c.ctas_per_sm;
  const double full_groups = (double)(int64_t)(per_sm / cps);
  const double rem = per_sm - full_groups * cps;  // tiles of the partial group (0 .. cps-1)
  // `efficiency` is the measured fraction of the arithmetic pipe's peak with the SM fully populated by this
  // variant; with fewer resident warps the pipe waits on latencies.  Measured with the 64 x 64 DMMA tile and
  // cp.async staging: 4 warps on an SM reach about 0.6 of that, 8 warps 0.85, 16 warps all of it -- fitted by
  // 1 - exp(-w/4.3).  TMA staging (no staging instructions, no CTA-wide barrier) loses less: 1 - exp(-w/3.3).
  const double efold = c.extra_fixed_clks > 0.0 ? 3.3 : 4.3;
  const double w_full = cps * c.threads / 32.0;
  auto occupancy = [&](double ctas) {
    return (1.0 - exp(-(ctas * c.threads / 32.0) / efold)) / (1.0 - exp(-w_full / efold));
  };
  // feed: bytes of A and B a tile pulls through L2; epilogue: C read + write at the SM's share of HBM bandwidth
  const double t_feed = (double)(c.bm + c.bn) * c.bk * kt * elem_bytes / r.l2_bytes_per_clk;
  const double t_epi = 2.0 * c.bm * c.bn * elem_bytes / r.hbm_bytes_per_clk;
  const double t_fixed = r.tile_fixed_clks + c.extra_fixed_clks + t_epi;
  auto tile_clks = [&](double occ) {
    const double t_math = fma_tile / (r.fma_per_clk * c.efficiency * occ);
    const double t_main = t_math > t_feed ? t_math : t_feed;
    return (t_main > t_epi ? t_main : t_epi) + c.per_tile_extra_clks;
  };
  if (per_sm < 2.0) return per_sm * (tile_clks(occupancy(1.0)) + t_fixed);  // nothing overlaps the fixed costs
  double total = full_groups * cps * tile_clks(1.0);
  if (rem > 0.0) {
    double occ = occupancy(rem);
    // Measured: the tiles of a launch that fits in one wave take about 8 % longer than the same tiles in a long
    // launch, where CTAs are dispatched one by one as others retire.
    if (full_groups == 0.0 && rem >= 3.0) occ *= 0.92;
    total += rem * tile_clks(occ);
  } else if (full_groups == 1.0 && tiles <= (double)sms * cps) {
    total /= 0.92;  // exactly one full wave: the same
  }
  // with >= 2 tiles per SM one tile's ramp-up and epilogue overlap another tile's main loop: paid once
  return total + t_fixed;
}

// Index of the candidate with the smallest estimate.
inline int select_tile(const TileChoice* cand, int count, int64_t m, int64_t n, int64_t k, int sms, int elem_bytes,
                       int64_t batch = 1) {
  int best = -1;
  double best_t = 0.0;
  for (int i = 0; i < count; ++i) {
    if (cand[i].explicit_only) continue;
    const double t = estimate_clks(cand[i], m, n, k, sms, elem_bytes, batch);
    if (best < 0 || t < best_t) best = i, best_t = t;
  }
  return best < 0 ? 0 : best;
}

}  // namespace b2
