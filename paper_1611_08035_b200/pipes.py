"""Measure the arithmetic-pipe rates the tile model needs (``python -m paper_1611_08035_b200.pipes``).

For every probe kind the C library offers, launch a grid that fills all SMs, read back the
per-CTA cycle counts and the CUDA-event time, and print multiply-adds per clock per SM, the
SM clock implied by (cycles / time) and TFLOP/s.  One JSON object per line.
"""
from __future__ import annotations

import argparse
import ctypes
import json

import torch

from . import binding

KINDS = {
    "dfma": 0,
    "ffma": 1,
    "dmma_m8n8k4": 2,
    "dmma_m16n8k4": 3,
    "dmma_m16n8k8": 4,
    "dmma_m16n8k16": 5,
    "ffma2": 6,
}


def probe(kind: str, threads_per_cta: int, ctas_per_sm: int, iters: int, repeats: int = 3) -> dict:
    lib = binding.lib()
    dev = torch.device("cuda", torch.cuda.current_device())
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    ctas = sms * ctas_per_sm
    scratch = torch.zeros(64 + 8 * ctas, dtype=torch.uint8, device=dev)
    per = ctypes.c_double(0.0)
    stream = torch.cuda.current_stream().cuda_stream
    best_ms, cycles = None, None
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rc = lib.b2_pipe_probe(KINDS[kind], threads_per_cta, ctas, iters, scratch.data_ptr(), scratch.numel(),
                               ctypes.byref(per), stream)
        e1.record()
        if rc != 0:
            raise RuntimeError(f"b2_pipe_probe failed: {binding.strerror(rc)}")
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if best_ms is None or ms < best_ms:
            best_ms = ms
            cycles = scratch[64:].view(torch.int64).double().mean().item()
    fma_total = float(threads_per_cta) * ctas * iters * per.value
    return {
        "kind": kind,
        "threads_per_cta": threads_per_cta,
        "ctas_per_sm": ctas_per_sm,
        "iters": iters,
        "ms": best_ms,
        "fma_per_clk_per_sm": fma_total / sms / cycles,
        "implied_sm_mhz": cycles / (best_ms * 1e-3) / 1e6,
        "tflops": 2.0 * fma_total / (best_ms * 1e-3) / 1e12,
    }


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=20000)
    ap.add_argument("--long-iters", type=int, default=0, help="also run each kind this long (sustained clocks)")
    args = ap.parse_args()
    for kind in KINDS:
        for tpc, cps in ((128, 1), (256, 1), (128, 2), (256, 2), (512, 2)):
            print(json.dumps(probe(kind, tpc, cps, args.iters)), flush=True)
        if args.long_iters:
            print(json.dumps(probe(kind, 256, 2, args.long_iters, repeats=1)), flush=True)


if __name__ == "__main__":
    main()
