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
    "mix_ffma2_8x8": 7,
    "mix_ffma2_16x8": 8,
    "mix_dmma_64x64": 9,
    "mix_ffma_8x8": 10,
    "mix_ffma2_4x4": 11,
    "mix_dfma_8x8": 12,
}
WITH_BARRIER = 0x100  # OR-ed into a mix kind: one CTA-wide barrier per slab
# residencies at which the GEMM kernels run each mix (CTAs of 128 threads per SM), plus one above and below
MIX_RESIDENCY = {"mix_ffma2_8x8": (2, 3, 4), "mix_ffma2_16x8": (1, 2), "mix_dmma_64x64": (2, 3, 4),
                 "mix_ffma_8x8": (3, 4), "mix_ffma2_4x4": (4, 8), "mix_dfma_8x8": (1, 2)}
MIX_THREADS = {"mix_ffma2_4x4": 64}


def probe(kind: str, threads_per_cta: int, ctas_per_sm: int, iters: int, repeats: int = 3,
          barrier: bool = False) -> dict:
    lib = binding.lib()
    code = KINDS[kind] | (WITH_BARRIER if barrier else 0)
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
        rc = lib.b2_pipe_probe(code, threads_per_cta, ctas, iters, scratch.data_ptr(), scratch.numel(),
                               ctypes.byref(per), stream)
        e1.record()
        if rc != 0:
            raise RuntimeError(f"b2_pipe_probe failed: {binding.strerror(rc)}")
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if best_ms is None or ms < best_ms:
            best_ms = ms
            # the slowest CTA: CTAs that share an SM do not get equal shares of it, so the early finishers'
            # cycle counts understate the time the work took
            cycles = scratch[64:].view(torch.int64).double().max().item()
    fma_total = float(threads_per_cta) * ctas * iters * per.value
    return {
        "kind": kind + ("+barrier" if barrier else ""),
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
        if kind in MIX_RESIDENCY:
            for cps in MIX_RESIDENCY[kind]:
                for barrier in (False, True):
                    print(json.dumps(probe(kind, MIX_THREADS.get(kind, 128), cps, max(1, args.iters // 16), barrier=barrier)), flush=True)
            continue
        for tpc, cps in ((128, 1), (256, 1), (128, 2), (256, 2), (512, 2)):
            print(json.dumps(probe(kind, tpc, cps, args.iters)), flush=True)
        if args.long_iters:
            print(json.dumps(probe(kind, 256, 2, args.long_iters, repeats=1)), flush=True)


if __name__ == "__main__":
    main()
