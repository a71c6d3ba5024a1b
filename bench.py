#!/usr/bin/env python
"""Benchmark of the GEMM hot path: one JSON line on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one pass of the whole hot path (tile loop, staging, micro-kernel, fringe handling,
fused epilogue -- one kernel launch) over the headline workload: fp64 GEMM, column-major NN,
m = n = k = 8192, alpha = 1.5, beta = 0.5, operands i.i.d. uniform[-1, 1) from a seed.
`value` is GFLOP/s (2*m*n*k flops per step) with the operands resident in HBM; `e2e` is the
same metric through the host-buffer C entry point with the host<->device copies inside the
timed region.  With N > 1 every rank runs the same workload on its own GPU (independent
problems, no data-path collective): weak scaling, time = max over ranks.

`--impl reference` times the CPU oracle (plain triple loop) on a bounded column sample of the
same workload on the host cores; it is a deliberately slow baseline.

`--case ...` runs ONE problem a few times and prints its time (a small driver for profilers and
quick timing; see `case_main`):

    python bench.py --case --dtype d -m 4096 -n 4096 -k 4096 [--transa T] [--pad] [--variant 4] [--iters 2]
    python bench.py --case --dtype tf32x1 -m 8192 -n 8192 -k 8192
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

WORKLOAD = dict(name="dgemm_nn_8192", transa="N", transb="N", m=8192, n=8192, k=8192, alpha=1.5, beta=0.5,
                dist="uniform", seed=2013)
# FP64 peak: 148 SMs x 64 FP64 multiply-adds per clock per SM (DFMA and DMMA probes both measure 64.0) x 2 flops
# x 1.965 GHz maximum SM clock.  FP32: 128 FFMA per clock per SM.
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
# ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch of the headline kernel, with the kernel it was
# captured on: written next to the profile summary, read here, and dropped when the selector launches another kernel.
TRAFFIC_FILE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "profiles", "dgemm_nn_8192_dram_traffic.json")
ORACLE_SAMPLE_COLUMNS = 96
OTHERS_LAUNCHES = 20  # timed launches per configuration (after 3 warm-ups); median and minimum are reported


def headline_traffic(kernel_name: str):
    """(bytes, note) of the recorded DRAM traffic of one headline launch; bytes is None when the record is
    missing or belongs to another kernel."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
    except (OSError, ValueError):
        return None, "no traffic record"
    if rec.get("kernel") != kernel_name:
        return None, f"traffic record is for kernel {rec.get('kernel')}, this run launched {kernel_name}"
    return float(rec["dram_bytes_per_launch"]), f"ncu capture of {rec['kernel']} ({rec.get('source', '')})"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None
        self.window = [None, None]  # host times of the first and last timed event

    def mark_begin(self):
        self.window[0] = time.perf_counter()

    def mark_end(self):
        self.window[1] = time.perf_counter()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100", "-i",
                 str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        parsed = []
        for stamp, r in self.rows:
            if len(r) < 7:
                continue
            try:
                parsed.append((stamp, float(r[0]), float(r[1]), float(r[2]), r[3:7]))
            except ValueError:
                continue
        if not parsed:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # Samples under load are those printed between the first and the last timed event (a sample is printed
        # up to one period after it was taken, hence the slack); every one of them counts, so a down-clock that
        # affects any part of the timed region shows in the minimum and moves the median.
        t0, t1 = self.window
        inside = [p for p in parsed if t0 is not None and t1 is not None and t0 <= p[0] <= t1 + 0.15]
        how = "between the first and last timed event"
        if not inside:  # timed region shorter than the sampling period: the samples at the highest power draw
            top = max(p[3] for p in parsed)
            inside = [p for p in parsed if p[3] >= 0.8 * top]
            how = "no sample fell inside the timed region; samples at >= 80 % of the highest power draw"
        reasons = set()
        for p in inside:
            for name, flag in zip(names, p[4]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        clocks = [p[1] for p in inside]
        return {"sm_mhz": statistics.median(clocks), "sm_mhz_min": min(clocks), "sm_max_mhz": max(p[2] for p in parsed),
                "power_w_max": max(p[3] for p in inside), "samples": len(inside), "samples_total": len(parsed),
                "window": how, "reasons": sorted(reasons)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


def device_inputs(w, dtype, device, seed_shift=0):
    from paper_1611_08035_b200 import synth
    return synth.gemm_inputs(w["transa"], w["transb"], w["m"], w["n"], w["k"], w["dist"], w["seed"] + seed_shift,
                             dtype, device=device)


def time_steps(fn, steps, warmup, barrier, sampler=None):
    """W warm-up calls, then K timed calls bracketed by barrier + synchronize; per-step CUDA-event times (ms)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    events = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    if sampler is not None:
        sampler.mark_begin()
    events[0].record(stream)
    for i in range(steps):
        fn()
        events[i + 1].record(stream)
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.mark_end()
    barrier()
    total_ms = events[0].elapsed_time(events[-1])
    per_step = [events[i].elapsed_time(events[i + 1]) for i in range(steps)]
    return total_ms, per_step


def timed_launches(fn, flops, iters=OTHERS_LAUNCHES, warm=3):
    """`warm` untimed calls, then `iters` back-to-back calls with a CUDA event between each; returns
    {"gflops": from the median time, "gflops_best": from the shortest, "ms_median", "ms_min", "launches"}."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record()
    for i in range(iters):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]
    med, low = statistics.median(ms), min(ms)
    return {"gflops": round(flops / med / 1e6, 1), "gflops_best": round(flops / low / 1e6, 1),
            "ms_median": round(med, 4), "ms_min": round(low, 4), "launches": iters}


def quick_gflops(fn, flops, iters=OTHERS_LAUNCHES, warm=3):
    return timed_launches(fn, flops, iters, warm)["gflops"]


def graph_gflops(fn, flops, launches=20, replays=10):
    """Throughput of `fn` replayed from a CUDA graph of `launches` back-to-back launches: the kernels' own time,
    without the host's per-launch cost (which bounds problems that take only a few microseconds)."""
    fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(launches):
            fn()
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return flops * launches * replays / (e0.elapsed_time(e1) * 1e-3) / 1e9


def oracle_check(fn, kind, ta, tb, m, n, k, alpha, beta, A, lda, B, ldb, C0, ldc):
    """One launch on a fresh copy of C against the CPU oracle (part of the CPU-baseline leg): largest observed
    |C - C_ref| / (2 k u S) over the compared columns, and the oracle's own time.  All of C for n <= 2048,
    otherwise first, last, both sides of a tile boundary and four seeded random columns."""
    import numpy as np
    from oracle import ref
    if n <= 2048:
        cols, sel = None, list(range(n))
    else:
        rng = np.random.default_rng(m + n + k)
        sel = sorted({0, n - 1, 63, 64} | {int(c) for c in rng.integers(0, n, size=4)})
        cols = sel
    Cd = C0.clone()
    fn(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, Cd, ldc)
    torch.cuda.synchronize()
    An, Bn, Cn = A.cpu().numpy(), B.cpu().numpy(), C0.cpu().numpy()
    want = Cn.copy()
    t0 = time.perf_counter()
    ref.ref_gemm(ta, tb, m, n, k, alpha, An, lda, Bn, ldb, beta, want, ldc, cols=cols)
    secs = time.perf_counter() - t0
    _, S = ref.ref_gemm_hi(ta, tb, m, n, k, alpha, An, lda, Bn, ldb, beta, Cn, ldc, cols=cols)
    got = Cd.cpu().numpy().reshape(n, ldc)[sel, :m].astype(np.float64)
    w = want.reshape(n, ldc)[sel, :m].astype(np.float64)
    u = 2.0 ** -53 if kind == "d" else 2.0 ** -24
    bound = 2.0 * k * u * S.reshape(n, m)[sel, :]
    ratio = float((np.abs(got - w) / np.maximum(bound, 1e-300)).max())
    return {"max_error_over_bound": round(ratio, 4), "columns": len(sel), "oracle_seconds": round(secs, 3),
            "oracle_gflops": round(2.0 * m * len(sel) * k / secs / 1e9, 2), "oracle_threads": ref.num_threads()}


def other_configs(b2, device, with_oracle=True):
    """The remaining benchmark configurations: OTHERS_LAUNCHES timed launches each after three warm-ups (median
    and best), C reused in place (alpha = 1.5, beta = 0.5 keeps it bounded; the rank-k updates grow it linearly, far
    from overflow); with `with_oracle`, one extra launch per real configuration is checked against the CPU oracle."""
    from paper_1611_08035_b200 import synth
    out = []

    def real(kind, ta, tb, m, n, k, alpha, beta, dist, seed, pad, label):
        dt = torch.float64 if kind == "d" else torch.float32
        (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
        lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(m)) if pad else (None, None, None)
        A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, dist, seed, dt, *lds, device=device)
        fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
        check = oracle_check(fn, kind, ta, tb, m, n, k, alpha, beta, A, lda, B, ldb, C, ldc) if with_oracle else None
        t = timed_launches(lambda: fn(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc), 2.0 * m * n * k)
        g = t["gflops"]
        peak = FP64_PEAK_TFLOPS if kind == "d" else FP32_PEAK_TFLOPS
        cfg = json.loads(b2.b2_gemm_query_config(0 if kind == "d" else 1, ta, tb, m, n, k, lda, ldb, ldc))
        if kind == "s" and beta in (0.0, 1.0) and k <= 1024 and not pad and (ta, tb) != ("T", "N") \
                and 2 * (-(-m // 128)) * (-(-n // 128)) >= 3 * torch.cuda.get_device_properties(device).multi_processor_count:
            # the query answers for a general beta; such an update goes to the TMA-staged kernel (b2gemm.h)
            cfg["name"] = [b2.b2_variant_name(1, v) for v in range(b2.b2_variant_count(1))
                           if "tma" in b2.b2_variant_name(1, v)][0]
            cfg["k_split"] = 1
        row = {"workload": label, "gflops": g, "gflops_best": t["gflops_best"], "ms_median": t["ms_median"],
               "launches": t["launches"], "frac_of_peak": round(g / 1e3 / peak, 4),
               "kernel": cfg["name"] + (f"/k_split {cfg['k_split']}" if cfg["k_split"] > 1 else "")}
        if check is not None:
            row["oracle"] = check
        if max(m, n, k) <= 1024 and not pad:  # microsecond-scale problems: also the kernel time without launch cost
            gg = graph_gflops(lambda: fn(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc), 2.0 * m * n * k)
            row["gflops_graph_replay"] = round(gg, 1)
            row["frac_of_peak_graph_replay"] = round(gg / 1e3 / peak, 4)
        if label.startswith("rank_k"):
            ms = 2.0 * m * n * k / g / 1e6
            row["hbm_gbs"] = round((2.0 * m * n + (m + n) * k) * (8 if kind == "d" else 4) / (ms * 1e-3) / 1e9, 1)
        out.append(row)
        del A, B, C

    real("d", "N", "N", 256, 256, 256, 1.0, 0.0, "uniform", 0, False, "dgemm_nn_256")
    for s in (512, 1024, 2048, 4096):
        real("d", "N", "N", s, s, s, 1.5, 0.5, "uniform", 2000, False, f"dgemm_nn_{s}")
    for s in (512, 1024, 2048, 4096, 8192):
        real("s", "N", "N", s, s, s, 1.5, 0.5, "uniform", 2100, False, f"sgemm_nn_{s}")
    for kind in "ds":  # the other three transpose combinations of the 4096^3 problem
        for ta, tb in (("N", "T"), ("T", "N"), ("T", "T")):
            real(kind, ta, tb, 4096, 4096, 4096, 1.5, 0.5, "uniform", 2200, False,
                 f"{kind}gemm_{ta.lower()}{tb.lower()}_4096")
    for k in (64, 128, 256):
        real("d", "N", "N", 16384, 16384, k, -1.0, 1.0, "normal", 3000 + k, False, f"rank_k_dgemm_16384_k{k}")
    real("s", "N", "N", 16384, 16384, 64, -1.0, 1.0, "normal", 3100, False, "rank_k_sgemm_16384_k64")
    for kind in "ds":
        for ta in "NT":
            for tb in "NT":
                real(kind, ta, tb, 1001, 999, 1003, 0.7, -0.3, "uniform", 4000, True,
                     f"{kind}gemm_{ta.lower()}{tb.lower()}_1001x999x1003_ld1027")
    # level-3 consumers of the kernel: symmetric rank-k update (n*n*k flops: half of the GEMM) and a strided batch
    for n_, k_ in ((8192, 8192), (16384, 256)):
        A = synth.matrix(n_, k_, n_, "uniform", 7000, torch.float64, device=device)
        C = synth.matrix(n_, n_, n_, "uniform", 7001, torch.float64, device=device)
        g = quick_gflops(lambda: b2.b2_syrk("L", "N", n_, k_, -1.0, A, n_, 1.0, C, n_), 1.0 * n_ * n_ * k_)
        out.append({"workload": f"dsyrk_ln_n{n_}_k{k_}", "gflops": round(g, 1), "frac_of_peak": round(g / 1e3 / FP64_PEAK_TFLOPS, 4),
                    "note": "n*n*k flops (stored triangle only)"})
        del A, C
    bm, bb = 512, 64
    A = synth.matrix(bm, bm * bb, bm, "uniform", 7100, torch.float64, device=device)
    B = synth.matrix(bm, bm * bb, bm, "uniform", 7101, torch.float64, device=device)
    C = synth.matrix(bm, bm * bb, bm, "uniform", 7102, torch.float64, device=device)
    g = quick_gflops(lambda: b2.b2_gemm_strided_batched("N", "N", bm, bm, bm, 1.5, A, bm, bm * bm, B, bm, bm * bm, 0.5, C,
                                                        bm, bm * bm, bb), 2.0 * bm ** 3 * bb)
    out.append({"workload": f"dgemm_strided_batched_{bb}x{bm}^3", "gflops": round(g, 1),
                "frac_of_peak": round(g / 1e3 / FP64_PEAK_TFLOPS, 4)})
    del A, B, C
    # fp32 on the tensor cores in TF32: reported separately, with the error each variant is specified with
    for terms, err in ((1, "2^-10 * S"), (3, "fp32 level: (2^-21 + 2(3k+2) 2^-24) * S")):
        for s in (4096, 8192):
            A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", s, s, s, "uniform", 2100, torch.float32, device=device)
            ws = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(terms, s, s, s), dtype=torch.uint8, device=device)
            g = quick_gflops(lambda: b2.b2_sgemm_tf32(terms, "N", "N", s, s, s, 1.5, A, lda, B, ldb, 0.5, C, ldc, ws),
                             2.0 * s * s * s)
            out.append({"workload": f"sgemm_tf32x{terms}_nn_{s}", "gflops": round(g, 1),
                        "note": "tcgen05 kind::tf32, not FP32-FMA arithmetic; 2*m*n*k flops counted once; packing "
                                "included", "error_bound_vs_fp32": err})
            del A, B, C, ws
    m = n = k = 4096
    A = synth.matrix(m, k, m, "uniform", 5000, torch.complex128, device=device)
    B = synth.matrix(k, n, k, "uniform", 5002, torch.complex128, device=device)
    C = torch.zeros(m * n, dtype=torch.complex128, device=device)
    ws = torch.empty(b2.b2_zgemm4m_workspace_bytes("N", "N", m, n, k), dtype=torch.uint8, device=device)
    t = timed_launches(lambda: b2.b2_zgemm4m("N", "N", m, n, k, 1 + 0.5j, A, m, B, k, 0j, C, m, ws), 8.0 * m * n * k)
    out.append({"workload": "zgemm4m_nn_4096", "gflops": t["gflops"], "gflops_best": t["gflops_best"],
                "ms_median": t["ms_median"], "launches": t["launches"],
                "frac_of_peak": round(t["gflops"] / 1e3 / FP64_PEAK_TFLOPS, 4),
                "note": "8*m*n*k flops; error bound with the 4M factor: 2(2k+4) u S per component"})
    # small m*n, long k: split-K against the plain kernel
    sm, sn, sk = 256, 256, 65536
    As = synth.matrix(sm, sk, sm, "uniform", 71, torch.float64, device=device)
    Bs = synth.matrix(sk, sn, sk, "uniform", 72, torch.float64, device=device)
    Cs = torch.zeros(sm * sn, dtype=torch.float64, device=device)
    wss = torch.empty(max(256, b2.b2_gemm_splitk_workspace_bytes(torch.float64, sm, sn, sk, 0)), dtype=torch.uint8,
                      device=device)
    g0 = quick_gflops(lambda: b2.b2_dgemm("N", "N", sm, sn, sk, 1.0, As, sm, Bs, sk, 0.0, Cs, sm), 2.0 * sm * sn * sk)
    g1 = quick_gflops(lambda: b2.b2_gemm_splitk("N", "N", sm, sn, sk, 1.0, As, sm, Bs, sk, 0.0, Cs, sm, 0, wss),
                      2.0 * sm * sn * sk)
    out.append({"workload": "dgemm_splitk_256x256x65536", "gflops": round(g1, 1), "plain_kernel_gflops": round(g0, 1),
                "splits": b2.b2_gemm_splitk_auto(sm, sn, sk), "frac_of_peak": round(g1 / 1e3 / FP64_PEAK_TFLOPS, 4)})
    del As, Bs, Cs, wss
    del ws
    ws = torch.empty(b2.b2_zgemm3m_workspace_bytes("N", "N", m, n, k), dtype=torch.uint8, device=device)
    g = quick_gflops(lambda: b2.b2_zgemm3m("N", "N", m, n, k, 1 + 0.5j, A, m, B, k, 0j, C, m, ws), 8.0 * m * n * k)
    out.append({"workload": "zgemm3m_nn_4096", "gflops": round(g, 1),
                "note": "8*m*n*k flops counted although 3M executes 6*m*n*k: the figure may exceed the FP64 peak",
                "frac_of_peak_executed": round(0.75 * g / 1e3 / FP64_PEAK_TFLOPS, 4)})
    return out


def oracle_sample_gflops(w, ncols, repeats=1):
    """Time the oracle on `ncols` seeded columns of the workload; returns (GFLOP/s, threads, seconds per call)."""
    import numpy as np
    from oracle import ref
    from paper_1611_08035_b200 import synth
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(w["transa"], w["transb"], w["m"], w["n"], w["k"], w["dist"], w["seed"],
                                               torch.float64)
    rng = np.random.default_rng(w["seed"])
    cols = sorted(int(c) for c in rng.choice(w["n"], size=ncols, replace=False))
    An, Bn, Cn = A.numpy(), B.numpy(), C.numpy()
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        ref.ref_gemm(w["transa"], w["transb"], w["m"], w["n"], w["k"], w["alpha"], An, lda, Bn, ldb, w["beta"], Cn,
                     ldc, cols=cols)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return 2.0 * w["m"] * ncols * w["k"] / best / 1e9, ref.num_threads(), best


def run_reference(args, rank):
    """The reference arm: the oracle as it stands on the host cores, bounded sample per step."""
    if rank != 0:
        return
    w = WORKLOAD
    ncols = ORACLE_SAMPLE_COLUMNS
    import numpy as np
    from oracle import ref
    from paper_1611_08035_b200 import synth
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(w["transa"], w["transb"], w["m"], w["n"], w["k"], w["dist"], w["seed"],
                                               torch.float64)
    cols = sorted(int(c) for c in np.random.default_rng(w["seed"]).choice(w["n"], size=ncols, replace=False))
    An, Bn, Cn = A.numpy(), B.numpy(), C.numpy()

    def step():
        ref.ref_gemm(w["transa"], w["transb"], w["m"], w["n"], w["k"], w["alpha"], An, lda, Bn, ldb, w["beta"], Cn, ldc,
                     cols=cols)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    gflops = 2.0 * w["m"] * ncols * w["k"] * args.steps / dt / 1e9
    sample = f"{ncols} seeded columns of C (all {w['m']} rows, full k) per step"
    line = {
        "impl": "reference", "metric": "DGEMM GFLOP/s (2*m*n*k flops)", "value": gflops, "unit": "GFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w["name"], "m": w["m"], "n": w["n"], "k": w["k"], "alpha": w["alpha"],
                   "beta": w["beta"], "layout": "column-major NN", "sample": sample},
        "cpu_baseline": {"value": gflops, "unit": "GFLOP/s", "cores": ref.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": gflops, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def case_main(argv):
    """`bench.py --case ...`: one problem, seeded inputs on the device, `--warmup` untimed and `--iters` timed calls,
    one JSON line with the CUDA-event time per call.  For profilers and quick timing (every kernel of the call is
    the product's own; nothing else is launched inside the timed region)."""
    from paper_1611_08035_b200 import binding as b2, synth
    ap = argparse.ArgumentParser(prog="bench.py --case")
    ap.add_argument("--dtype", choices=["d", "s", "z", "tf32x1", "tf32x3"], default="d")
    ap.add_argument("--transa", default="N")
    ap.add_argument("--transb", default="N")
    ap.add_argument("-m", type=int, default=4096)
    ap.add_argument("-n", type=int, default=4096)
    ap.add_argument("-k", type=int, default=4096)
    ap.add_argument("--alpha", type=float, default=1.5)
    ap.add_argument("--beta", type=float, default=0.5)
    ap.add_argument("--dist", default="uniform")
    ap.add_argument("--pad", action="store_true", help="leading dimensions = next multiple of 32, plus 3")
    ap.add_argument("--variant", type=int, default=None, help="explicit kernel variant (+256*s: k split over s CTAs)")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --case needs a CUDA device")
    b2.lib()
    dt = {"d": torch.float64, "s": torch.float32, "z": torch.complex128, "tf32x1": torch.float32,
          "tf32x3": torch.float32}[a.dtype]
    (ra, _), (rb, _) = synth.operand_shapes(a.transa, a.transb, a.m, a.n, a.k)
    lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(a.m)) if a.pad else (None, None, None)
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(a.transa, a.transb, a.m, a.n, a.k, a.dist, 1, dt, *lds, device="cuda")
    tr = (a.transa, a.transb, a.m, a.n, a.k)
    if a.dtype == "z":
        ws = torch.empty(b2.b2_zgemm4m_workspace_bytes(*tr), dtype=torch.uint8, device="cuda")

        def run():
            b2.b2_zgemm4m(*tr, complex(a.alpha, 0.5), A, lda, B, ldb, complex(a.beta), C, ldc, ws)
    elif a.dtype.startswith("tf32"):
        terms = int(a.dtype[-1])
        ws = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(terms, a.m, a.n, a.k), dtype=torch.uint8, device="cuda")

        def run():
            b2.b2_sgemm_tf32(terms, *tr, a.alpha, A, lda, B, ldb, a.beta, C, ldc, ws)
    else:
        fn = b2.b2_dgemm if a.dtype == "d" else b2.b2_sgemm

        def run():
            fn(*tr, a.alpha, A, lda, B, ldb, a.beta, C, ldc, variant=a.variant)

    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    flops = (8.0 if a.dtype == "z" else 2.0) * a.m * a.n * a.k
    kernel = None
    if a.dtype in ("d", "s") and a.variant is None:
        kernel = json.loads(b2.b2_gemm_query_config(0 if a.dtype == "d" else 1, *tr, lda, ldb, ldc))["name"]
    elif a.dtype in ("d", "s"):
        kernel = b2.b2_variant_name(0 if a.dtype == "d" else 1, a.variant & 255)
    print(json.dumps({"dtype": a.dtype, "trans": a.transa + a.transb, "m": a.m, "n": a.n, "k": a.k, "variant": a.variant,
                      "kernel": kernel, "ms_per_launch": ms, "gflops": flops / ms / 1e6,
                      "device_status": b2.b2_device_status()}))


def main():
    if "--case" in sys.argv[1:]:
        case_main([x for x in sys.argv[1:] if x != "--case"])
        return
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["b2gemm", "reference"], default="b2gemm")
    ap.add_argument("--no-others", action="store_true", help="skip the remaining configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.warmup < 3:
        args.warmup = 3
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")

    from paper_1611_08035_b200 import binding as b2
    b2.lib()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)
        sync_t = torch.zeros(1, device=device)

        def barrier():
            dist.all_reduce(sync_t)
            torch.cuda.synchronize()
    else:
        dist = None

        def barrier():
            return None

    w = WORKLOAD
    m, n, k = w["m"], w["n"], w["k"]
    flops = 2.0 * m * n * k
    from paper_1611_08035_b200 import replicas
    A, lda, B, ldb, C, ldc = device_inputs(w, torch.float64, device, seed_shift=replicas.rank_seed(0, rank))

    def step():
        b2.b2_dgemm(w["transa"], w["transb"], m, n, k, w["alpha"], A, lda, B, ldb, w["beta"], C, ldc)

    sampler = ClockSampler(visible_gpu_index(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    total_ms, per_step = time_steps(step, args.steps, args.warmup, barrier, sampler if rank == 0 else None)
    clocks = sampler.stop() if rank == 0 else None
    value, total_ms = replicas.aggregate_gflops(flops, args.steps, total_ms, world, dist, device)
    kernel_ms = statistics.mean(per_step)

    # end to end: host buffers in, result back in host memory, through the host-buffer C entry point
    Ah, Bh, Ch = (x.cpu().pin_memory() for x in (A, B, C))
    ws = torch.empty(b2.b2_gemm_host_workspace_bytes(0, w["transa"], w["transb"], m, n, k), dtype=torch.uint8,
                     device=device)

    def e2e_step():
        b2.b2_dgemm_host(w["transa"], w["transb"], m, n, k, w["alpha"], Ah, lda, Bh, ldb, w["beta"], Ch, ldc, ws)

    e2e_steps = max(2, min(args.steps, 5))
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()  # synchronises the stream before returning
    e2e_s = time.perf_counter() - t0
    e2e_value, _ = replicas.aggregate_gflops(flops, e2e_steps, e2e_s * 1e3, world, dist, device)
    elem = 8
    h2d = (m * k + k * n + m * n) * elem
    d2h = m * n * elem
    del Ah, Bh, Ch, ws

    others = None
    cpu_baseline = None
    if rank == 0 and world == 1:
        if not args.no_others:
            del A, B, C
            torch.cuda.empty_cache()
            others = other_configs(b2, device, with_oracle=not args.no_cpu_baseline)
        if not args.no_cpu_baseline:
            g, cores, secs = oracle_sample_gflops(w, ORACLE_SAMPLE_COLUMNS)
            cpu_baseline = {"value": g, "unit": "GFLOP/s", "cores": cores, "kind": "oracle",
                            "sample": f"{ORACLE_SAMPLE_COLUMNS} seeded columns of C (all {m} rows, full k) of the "
                                      f"same workload, one call, {secs:.1f} s",
                            "per_config": "others[*].oracle: the oracle's time and the largest error / bound of one "
                                          "launch per real configuration (all of C for n <= 2048, a column sample "
                                          "above)"}

    if rank == 0:
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        cfg = json.loads(b2.b2_gemm_query_config(0, w["transa"], w["transb"], m, n, k, lda, ldb, ldc))
        traffic, traffic_note = headline_traffic(cfg["name"])
        line = {
            "metric": "DGEMM GFLOP/s (2*m*n*k flops)", "value": value, "unit": "GFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w["name"], "m": m, "n": n, "k": k, "alpha": w["alpha"], "beta": w["beta"],
                       "layout": "column-major NN, lda=ldb=ldc=8192", "kernel": cfg["name"],
                       "l2": "operands (3 x 512 MiB) are larger than the 126 MB L2; no flush between steps",
                       "multi_gpu": "independent replicas, one problem per GPU, no collective"},
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
            "frac_of_fp64_peak": value / world / 1e3 / FP64_PEAK_TFLOPS,
            "frac_of_fp64_peak_at_observed_clock": (
                value / world / 1e3 / (FP64_PEAK_TFLOPS * clocks["sm_mhz"] / 1965.0)
                if clocks and clocks.get("sm_mhz") else None),
            "fp64_peak_tflops": FP64_PEAK_TFLOPS,
            "fp64_peak_source": "148 SMs x 64 FP64 FMA/clk/SM (measured by the DFMA and DMMA probes) x 2 x 1.965 GHz",
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "GFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": args.steps,
            "roofline": {"bound": "alu", "achieved": achieved, "peak": FP64_PEAK_TFLOPS, "unit": "TFLOP/s",
                         "frac": achieved / FP64_PEAK_TFLOPS, "traffic": traffic, "traffic_source": traffic_note,
                         "peak_source": "derived: FP64 pipe, 148 SMs x 64 FMA/clk x 2 x 1.965 GHz (see "
                                        "fp64_peak_source); HBM is not the bound at k = 8192"},
            "cpu_baseline": cpu_baseline,
        }
        if others is not None:
            line["others"] = others
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
