// C-ABI entry points of the analytical model (host-only; nothing is launched).
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

extern "C" int b2_model_predict_variant(int dtype, int variant, double* fraction, char* json_out, size_t cap) {
  using namespace b2;
  using namespace b2::model;
  if (dtype != B2_F64 && dtype != B2_F32) return -1;
  if (variant < 0 || variant >= b2_variant_count(dtype)) return -2;
  if (!fraction) return -3;
  const VariantInfo& vi = dtype == B2_F64 ? f64_variant_info(variant) : f32_variant_info(variant);
  int kind;
  if (strncmp(vi.micro, "dmma", 4) == 0) kind = MK_DMMA;
  else if (strcmp(vi.micro, "dfma") == 0) kind = MK_DFMA;
  else if (strcmp(vi.micro, "ffma2") == 0) kind = MK_FFMA2;
  else kind = MK_FFMA;
  const int warps = vi.threads / 32;
  // warp tile: DMMA variants split the CTA tile 2 x (warps/2); FMA variants cover 8 x 4 lanes of tm x tn blocks
  const int wtm = kind == MK_DMMA ? vi.bm / 2 : 8 * vi.tm;
  const int wtn = kind == MK_DMMA ? vi.bn / (warps / 2) : 4 * vi.tn;
  const int elem = dtype == B2_F64 ? 8 : 4;
  const int staging = (vi.bm + vi.bn) * vi.bk * elem / 16 / vi.threads;  // 16-byte chunks per thread per slab
  const WarpMix mix = warp_mix(kind, wtm, wtn, staging, vi.bk);
  *fraction = predicted_fraction(mix, dtype == B2_F64);
  if (json_out) {
    double rate[NPIPES];
    sm_rates(rate);
    char buf[768];
    const int len = snprintf(
        buf, sizeof(buf),
        "{\"variant\": \"%s\", \"micro_kernel\": \"%s\", \"warp_tile\": [%d, %d], \"jobs_per_k\": {\"issue\": %.4f, "
        "\"fp64\": %.4f, \"tensor64\": %.4f, \"fp32\": %.4f, \"lsu\": %.4f}, \"clocks_per_k\": {\"issue\": %.4f, "
        "\"fp64\": %.4f, \"tensor64\": %.4f, \"fp32\": %.4f, \"lsu\": %.4f}, \"predicted_fraction\": %.4f, "
        "\"measured_fraction\": %.4f}",
        vi.name, vi.micro, wtm, wtn, mix.jobs[ISSUE], mix.jobs[FP64], mix.jobs[TENSOR64], mix.jobs[FP32],
        mix.jobs[LSU], mix.jobs[ISSUE] / rate[ISSUE], mix.jobs[FP64] / rate[FP64], mix.jobs[TENSOR64] / rate[TENSOR64],
        mix.jobs[FP32] / rate[FP32], mix.jobs[LSU] / rate[LSU], *fraction, vi.efficiency);
    if (len < 0 || (size_t)len + 1 > cap) return B2_ERR_WORKSPACE;
    memcpy(json_out, buf, (size_t)len + 1);
  }
  return B2_OK;
}
