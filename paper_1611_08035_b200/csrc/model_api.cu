// C-ABI entry points of the analytical model (host-only; nothing is launched).
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "b2gemm.h"
#include "gemm_launch.cuh"
#include "queue_model.h"

extern "C" double b2_model_throughput(int npipes, const double* rate, const double* jobs) {
  return b2::model::throughput(npipes, rate, jobs);
}

extern "C" double b2_model_stalled_throughput(double jobs, int n_dependent, double latency) {
  return b2::model::stalled_throughput(jobs, n_dependent, latency);
}

extern "C" int b2_model_register_updates(int r_total, int mr, int nr, int v, int r_a, int r_r, int* n_updates) {
  if (!n_updates) return -7;
  bool ok = false;
  const int n = b2::model::register_updates(r_total, mr, nr, v, r_a, r_r, &ok);
  if (!ok) return -1;
  *n_updates = n;
  return B2_OK;
}

namespace b2 {

// Limits of the current device's SMs (queried once; the B200 values when no device can be asked).
model::SmLimits sm_limits() {
  static const model::SmLimits cached = [] {
    model::SmLimits lim;
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return lim;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxRegistersPerMultiprocessor, dev) == cudaSuccess && v > 0) lim.regs_per_sm = v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) == cudaSuccess && v > 0) lim.smem_per_sm = v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxThreadsPerMultiProcessor, dev) == cudaSuccess && v > 0) lim.max_warps_per_sm = v / 32;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxBlocksPerMultiprocessor, dev) == cudaSuccess && v > 0) lim.max_ctas_per_sm = v;
    return lim;
  }();
  return cached;
}

namespace {
int kind_of(const VariantInfo& vi) {
  if (strncmp(vi.micro, "dmma", 4) == 0) return model::MK_DMMA;
  if (strcmp(vi.micro, "dfma") == 0) return model::MK_DFMA;
  if (strncmp(vi.micro, "ffma2", 5) == 0) return model::MK_FFMA2;
  return model::MK_FFMA;
}
}  // namespace

// The candidate a built variant corresponds to: its warp tile, warp grid, slab depth and ring stages.
model::SmCandidate candidate_of(const VariantInfo& vi) {
  model::SmCandidate c;
  c.kind = kind_of(vi);
  // the persistent kernel's groups are four-warp CTAs in all but name; its extra warpgroup moves no data
  const int warps = strcmp(vi.micro, "dmma_ws") == 0 ? 4 : vi.threads / 32;
  if (c.kind == model::MK_DMMA) {  // DMMA variants split the CTA tile 2 x (warps/2)
    c.warps_m = 2, c.warps_n = warps / 2;
    c.wtm = vi.bm / c.warps_m, c.wtn = vi.bn / c.warps_n;
  } else {  // FMA variants: a warp covers 8 x 4 lanes of tm x tn blocks
    c.wtm = 8 * vi.tm, c.wtn = 4 * vi.tn;
    c.warps_m = vi.bm / c.wtm, c.warps_n = vi.bn / c.wtn;
  }
  c.bk = vi.bk, c.stages = vi.stages;
  c.tma = strcmp(vi.micro, "dmma_tma") == 0 || strcmp(vi.micro, "dmma_ws") == 0 || strcmp(vi.micro, "ffma2_tma") == 0;
  return c;
}

// Model prediction for a built variant at the residency it is launched with.
model::SmPrediction predict_variant(int dtype, int variant) {
  const VariantInfo& vi = dtype == B2_F64 ? f64_variant_info(variant) : f32_variant_info(variant);
  model::SmLimits lim = sm_limits();
  lim.max_ctas_per_sm = strcmp(vi.micro, "dmma_ws") == 0 ? 3 : vi.ctas_per_sm;  // as launched, not as it could be
  return model::predict(candidate_of(vi), lim, dtype == B2_F64 ? 8 : 4);
}

}  // namespace b2

extern "C" int b2_model_predict_variant(int dtype, int variant, double* fraction, char* json_out, size_t cap) {
  using namespace b2;
  using namespace b2::model;
  if (dtype != B2_F64 && dtype != B2_F32) return -1;
  if (variant < 0 || variant >= b2_variant_count(dtype)) return -2;
  if (!fraction) return -3;
  const VariantInfo& vi = dtype == B2_F64 ? f64_variant_info(variant) : f32_variant_info(variant);
  const SmCandidate c = candidate_of(vi);
  const SmPrediction pr = predict_variant(dtype, variant);
  const int elem = dtype == B2_F64 ? 8 : 4;
  const int threads = 32 * c.warps_m * c.warps_n;
  const int staging = (vi.bm + vi.bn) * vi.bk * elem / 16 / threads;  // 16-byte chunks per thread per slab
  const WarpMix mix = warp_mix(c.kind, c.wtm, c.wtn, c.tma ? 0 : (staging > 0 ? staging : 1), vi.bk);
  *fraction = pr.fraction;
  if (json_out) {
    double rate[NPIPES];
    sm_rates(rate);
    char buf[1024];
    const int len = snprintf(
        buf, sizeof(buf),
        "{\"variant\": \"%s\", \"micro_kernel\": \"%s\", \"warp_tile\": [%d, %d], \"jobs_per_k\": {\"issue\": %.4f, "
        "\"fp64\": %.4f, \"tensor64\": %.4f, \"fp32\": %.4f, \"lsu\": %.4f}, \"clocks_per_k\": {\"issue\": %.4f, "
        "\"fp64\": %.4f, \"tensor64\": %.4f, \"fp32\": %.4f, \"lsu\": %.4f}, \"pipe_fraction\": %.4f, "
        "\"feed_fraction\": %.4f, \"coverage\": %.4f, \"stall\": %.4f, \"registers\": %d, \"n_updates\": %d, \"ctas_per_sm\": %d, "
        "\"predicted_fraction\": %.4f, \"measured_fraction\": %.4f}",
        vi.name, vi.micro, c.wtm, c.wtn, mix.jobs[ISSUE], mix.jobs[FP64], mix.jobs[TENSOR64], mix.jobs[FP32],
        mix.jobs[LSU], mix.jobs[ISSUE] / rate[ISSUE], mix.jobs[FP64] / rate[FP64], mix.jobs[TENSOR64] / rate[TENSOR64],
        mix.jobs[FP32] / rate[FP32], mix.jobs[LSU] / rate[LSU], pr.pipe_fraction, pr.feed_fraction, pr.coverage, pr.stall,
        pr.regs_per_thread, pr.n_updates, pr.ctas_per_sm, pr.fraction, vi.efficiency);
    if (len < 0 || (size_t)len + 1 > cap) return B2_ERR_WORKSPACE;
    memcpy(json_out, buf, (size_t)len + 1);
  }
  return B2_OK;
}

// Section 5.1 ("A Work Flow for Kernel Generation"): enumerate the candidates, estimate each with the model,
// keep the best.  Candidates: micro-kernel kind x warp tile (the mr x nr of a warp) x warp grid x ring stages,
// kept when they fit the registers (Section 5's limit with at least two unit updates of fragments) and the
// shared memory of an SM.
extern "C" int b2_model_enumerate(int dtype, int top, char* json_out, size_t cap) {
  using namespace b2;
  using namespace b2::model;
  if (dtype != B2_F64 && dtype != B2_F32) return -1;
  if (top <= 0) return -2;
  if (!json_out) return -3;
  struct Row {
    SmCandidate c;
    SmPrediction p;
    const char* built;
  };
  static const int kWtm64[] = {16, 32, 64}, kWtn64[] = {8, 16, 32, 64};
  static const int kTm[] = {4, 8, 16}, kTn[] = {4, 8};
  static const int kGrid[][2] = {{1, 1}, {1, 2}, {2, 1}, {2, 2}, {1, 4}, {4, 1}, {2, 4}, {4, 2}};
  const int elem = dtype == B2_F64 ? 8 : 4;
  const SmLimits lim = sm_limits();
  static thread_local Row rows[2048];
  int n = 0;
  auto add = [&](int kind, int wtm, int wtn, bool tma) {
    for (const auto& gr : kGrid)
      for (int stages = 2; stages <= 4; ++stages) {
        if (n >= 2048) return;
        Row r;
        r.c = SmCandidate{kind, wtm, wtn, gr[0], gr[1], 16, stages, tma};
        if (wtm * gr[0] > 256 || wtn * gr[1] > 256) continue;
        r.p = predict(r.c, lim, elem);
        r.built = nullptr;
        if (r.p.feasible) rows[n++] = r;
      }
  };
  if (dtype == B2_F64) {
    for (int wtm : kWtm64)
      for (int wtn : kWtn64) {
        add(MK_DMMA, wtm, wtn, false);
        add(MK_DMMA, wtm, wtn, true);  // fragments read the source layout, so the tensor memory accelerator can stage
      }
    for (int tm : kTm)
      for (int tn : kTn) add(MK_DFMA, 8 * tm, 4 * tn, false);
  } else {
    for (int tm : kTm)
      for (int tn : kTn) {
        add(MK_FFMA2, 8 * tm, 4 * tn, false);  // the FMA kernels want both operands packed C-index-contiguous:
        add(MK_FFMA, 8 * tm, 4 * tn, false);   // staged (and transposed) by the warps themselves
      }
  }
  // which candidates exist as variants of the library
  const int nv = b2_variant_count(dtype);
  for (int v = 0; v < nv; ++v) {
    const VariantInfo& vi = dtype == B2_F64 ? f64_variant_info(v) : f32_variant_info(v);
    if (strcmp(vi.micro, "dmma_ws") == 0) continue;  // the tiles of dmma_tma_64x64, other scheduling
    const SmCandidate c = candidate_of(vi);
    for (int i = 0; i < n; ++i) {
      const SmCandidate& d = rows[i].c;
      if (d.kind == c.kind && d.wtm == c.wtm && d.wtn == c.wtn && d.warps_m == c.warps_m && d.warps_n == c.warps_n &&
          d.stages == c.stages && d.tma == c.tma)
        rows[i].built = vi.name;
    }
  }
  // rank: predicted fraction, ties to the larger CTA tile (fewer bytes per multiply-add), then fewer stages
  for (int i = 1; i < n; ++i) {
    Row r = rows[i];
    int j = i - 1;
    auto better = [](const Row& a, const Row& b) {
      if (fabs(a.p.fraction - b.p.fraction) > 1e-9) return a.p.fraction > b.p.fraction;
      if (a.p.bm * a.p.bn != b.p.bm * b.p.bn) return a.p.bm * a.p.bn > b.p.bm * b.p.bn;
      return a.c.stages < b.c.stages;
    };
    while (j >= 0 && better(r, rows[j])) rows[j + 1] = rows[j], --j;
    rows[j + 1] = r;
  }
  static const char* kKind[] = {"dmma", "dfma", "ffma", "ffma2"};
  size_t pos = 0;
  auto put = [&](const char* text) {
    const size_t len = strlen(text);
    if (pos + len + 1 > cap) return false;
    memcpy(json_out + pos, text, len + 1);
    pos += len;
    return true;
  };
  char buf[512];
  snprintf(buf, sizeof(buf), "{\"dtype\": \"%s\", \"candidates\": %d, \"ranked\": [", dtype == B2_F64 ? "f64" : "f32", n);
  if (!put(buf)) return B2_ERR_WORKSPACE;
  // the best `top`, and every built candidate wherever it ranks
  bool first = true;
  for (int i = 0; i < n; ++i) {
    if (i >= top && !rows[i].built) continue;
    const Row& r = rows[i];
    snprintf(buf, sizeof(buf),
             "%s{\"rank\": %d, \"kind\": \"%s\", \"warp_tile\": [%d, %d], \"warps\": [%d, %d], \"cta_tile\": [%d, %d], "
             "\"stages\": %d, \"tma\": %s, \"registers\": %d, \"n_updates\": %d, \"smem_bytes\": %d, \"ctas_per_sm\": %d, "
             "\"pipe_fraction\": %.4f, \"feed_fraction\": %.4f, \"coverage\": %.4f, \"stall\": %.4f, "
             "\"predicted_fraction\": %.4f, \"built_as\": %s%s%s}",
             first ? "" : ", ", i + 1, kKind[r.c.kind], r.c.wtm, r.c.wtn, r.c.warps_m, r.c.warps_n, r.p.bm, r.p.bn,
             r.c.stages, r.c.tma ? "true" : "false", r.p.regs_per_thread, r.p.n_updates, r.p.smem_bytes, r.p.ctas_per_sm, r.p.pipe_fraction,
             r.p.feed_fraction, r.p.coverage, r.p.stall, r.p.fraction, r.built ? "\"" : "", r.built ? r.built : "null",
             r.built ? "\"" : "");
    if (!put(buf)) return B2_ERR_WORKSPACE;
    first = false;
  }
  return put("]}") ? B2_OK : B2_ERR_WORKSPACE;
}
