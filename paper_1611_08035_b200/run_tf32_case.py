"""Run the TF32 tensor-core GEMM a few times (``python -m paper_1611_08035_b200.run_tf32_case --terms 1 -n 4096``).

A minimal driver for profilers: seeded square NN problem on the device, ``--iters`` calls, one JSON line."""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as b2, synth


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--terms", type=int, choices=[1, 3], default=1)
    ap.add_argument("-n", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=3)
    a = ap.parse_args()
    s = a.n
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", s, s, s, "uniform", 1, torch.float32, device="cuda")
    ws = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(a.terms, s, s, s), dtype=torch.uint8, device="cuda")
    b2.b2_sgemm_tf32(a.terms, "N", "N", s, s, s, 1.5, A, lda, B, ldb, 0.5, C, ldc, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        b2.b2_sgemm_tf32(a.terms, "N", "N", s, s, s, 1.5, A, lda, B, ldb, 0.5, C, ldc, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    print(json.dumps({"terms": a.terms, "n": s, "ms_per_call": ms, "gflops_2mnk": 2.0 * s ** 3 / ms / 1e6,
                      "status": b2.b2_device_status()}))


if __name__ == "__main__":
    main()
