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
# ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch of the headline kernel (13.09 GB + 0.534 GB,
# one-pass capture of the TMA-staged 64x64x16 kernel at 8192^3 with 12 tile rows per rasterisation group;
# summary under profiles/).
HEADLINE_DRAM_TRAFFIC_BYTES = 13.62e9
ORACLE_SAMPLE_COLUMNS = 96


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
            self.rows.append([c.strip() for c in line.split(",")])

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
        clocks, maxes, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                clocks.append(float(r[0])), maxes.append(float(r[1])), power.append(float(r[2]))
            except ValueError:
                continue
            for name, flag in zip(names, r[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if not clocks:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # samples under load: the upper half of the clock readings (idle samples before/after are dropped)
        loaded = sorted(clocks)[len(clocks) // 2:]
        return {"sm_mhz": statistics.median(loaded), "sm_max_mhz": max(maxes), "power_w_max": max(power),
                "samples": len(clocks), "reasons": sorted(reasons)}


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


def time_steps(fn, steps, warmup, barrier):
    """W warm-up calls, then K timed calls bracketed by barrier + synchronize; per-step CUDA-event times (ms)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    events = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    events[0].record(stream)
    for i in range(steps):
        fn()
        events[i + 1].record(stream)
    torch.cuda.synchronize()
    barrier()
    total_ms = events[0].elapsed_time(events[-1])
    per_step = [events[i].elapsed_time(events[i + 1]) for i in range(steps)]
    return total_ms, per_step


def quick_gflops(fn, flops, iters=3, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return flops * iters / (e0.elapsed_time(e1) * 1e-3) / 1e9


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


def other_configs(b2, device):
    """Throughput of the remaining benchmark configurations (few launches each); reported inside the JSON line."""
    from paper_1611_08035_b200 import synth
    out = []

    def real(kind, ta, tb, m, n, k, alpha, beta, dist, seed, pad, label):
        dt = torch.float64 if kind == "d" else torch.float32
        (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
        lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(m)) if pad else (None, None, None)
        A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, dist, seed, dt, *lds, device=device)
        fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
        g = quick_gflops(lambda: fn(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc), 2.0 * m * n * k)
        peak = FP64_PEAK_TFLOPS if kind == "d" else FP32_PEAK_TFLOPS
        row = {"workload": label, "gflops": round(g, 1), "frac_of_peak": round(g / 1e3 / peak, 4)}
        if max(m, n, k) <= 1024 and not pad:  # microsecond-scale problems: also the kernel time without launch cost
            gg = graph_gflops(lambda: fn(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc), 2.0 * m * n * k)
            row["gflops_graph_replay"] = round(gg, 1)
            row["frac_of_peak_graph_replay"] = round(gg / 1e3 / peak, 4)
        if label.startswith("rank_k"):
            ms = 2.0 * m * n * k / g / 1e6
            row["hbm_gbs"] = round((2.0 * m * n + (m + n) * k) * 8 / (ms * 1e-3) / 1e9, 1)
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
    g = quick_gflops(lambda: b2.b2_zgemm4m("N", "N", m, n, k, 1 + 0.5j, A, m, B, k, 0j, C, m, ws), 8.0 * m * n * k,
                     iters=2, warm=2)
    out.append({"workload": "zgemm4m_nn_4096", "gflops": round(g, 1), "frac_of_peak": round(g / 1e3 / FP64_PEAK_TFLOPS, 4)})
    # small m*n, long k: split-K against the plain kernel
    sm, sn, sk = 256, 256, 65536
    As = synth.matrix(sm, sk, sm, "uniform", 71, torch.float64, device=device)
    Bs = synth.matrix(sk, sn, sk, "uniform", 72, torch.float64, device=device)
    Cs = torch.zeros(sm * sn, dtype=torch.float64, device=device)
    wss = torch.empty(max(256, b2.b2_gemm_splitk_workspace_bytes(torch.float64, sm, sn, sk, 0)), dtype=torch.uint8,
                      device=device)
    g0 = quick_gflops(lambda: b2.b2_dgemm("N", "N", sm, sn, sk, 1.0, As, sm, Bs, sk, 0.0, Cs, sm), 2.0 * sm * sn * sk,
                      iters=5, warm=2)
    g1 = quick_gflops(lambda: b2.b2_gemm_splitk("N", "N", sm, sn, sk, 1.0, As, sm, Bs, sk, 0.0, Cs, sm, 0, wss),
                      2.0 * sm * sn * sk, iters=5, warm=2)
    out.append({"workload": "dgemm_splitk_256x256x65536", "gflops": round(g1, 1), "plain_kernel_gflops": round(g0, 1),
                "splits": b2.b2_gemm_splitk_auto(sm, sn, sk), "frac_of_peak": round(g1 / 1e3 / FP64_PEAK_TFLOPS, 4)})
    del As, Bs, Cs, wss
    del ws
    ws = torch.empty(b2.b2_zgemm3m_workspace_bytes("N", "N", m, n, k), dtype=torch.uint8, device=device)
    g = quick_gflops(lambda: b2.b2_zgemm3m("N", "N", m, n, k, 1 + 0.5j, A, m, B, k, 0j, C, m, ws), 8.0 * m * n * k,
                     iters=2, warm=2)
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


def main():
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
    total_ms, per_step = time_steps(step, args.steps, args.warmup, barrier)
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
            others = other_configs(b2, device)
        if not args.no_cpu_baseline:
            g, cores, secs = oracle_sample_gflops(w, ORACLE_SAMPLE_COLUMNS)
            cpu_baseline = {"value": g, "unit": "GFLOP/s", "cores": cores, "kind": "oracle",
                            "sample": f"{ORACLE_SAMPLE_COLUMNS} seeded columns of C (all {m} rows, full k) of the "
                                      f"same workload, one call, {secs:.1f} s"}

    if rank == 0:
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        cfg = json.loads(b2.b2_gemm_query_config(0, w["transa"], w["transb"], m, n, k, lda, ldb, ldc))
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
                         "frac": achieved / FP64_PEAK_TFLOPS, "traffic": HEADLINE_DRAM_TRAFFIC_BYTES,
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
