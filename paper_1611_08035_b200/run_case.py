"""Run one GEMM problem a few times (``python -m paper_1611_08035_b200.run_case ...``).

A minimal driver for profilers and quick timing: seeded inputs on the device, ``--warmup`` untimed
launches, ``--iters`` timed launches, one JSON line with the CUDA-event time per launch.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as b2, synth


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--dtype", choices=["d", "s", "z"], default="d")
    ap.add_argument("--transa", default="N")
    ap.add_argument("--transb", default="N")
    ap.add_argument("-m", type=int, default=4096)
    ap.add_argument("-n", type=int, default=4096)
    ap.add_argument("-k", type=int, default=4096)
    ap.add_argument("--alpha", type=float, default=1.5)
    ap.add_argument("--beta", type=float, default=0.5)
    ap.add_argument("--dist", default="uniform")
    ap.add_argument("--pad", action="store_true", help="leading dimensions = next multiple of 32, plus 3")
    ap.add_argument("--variant", type=int, default=None)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    a = ap.parse_args()
    dt = {"d": torch.float64, "s": torch.float32, "z": torch.complex128}[a.dtype]
    (ra, _), (rb, _) = synth.operand_shapes(a.transa, a.transb, a.m, a.n, a.k)
    lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(a.m)) if a.pad else (None, None, None)
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(a.transa, a.transb, a.m, a.n, a.k, a.dist, 1, dt, *lds, device="cuda")
    if a.dtype == "z":
        ws = torch.empty(b2.b2_zgemm4m_workspace_bytes(a.transa, a.transb, a.m, a.n, a.k), dtype=torch.uint8,
                         device="cuda")

        def run():
            b2.b2_zgemm4m(a.transa, a.transb, a.m, a.n, a.k, complex(a.alpha, 0.5), A, lda, B, ldb, complex(a.beta), C,
                          ldc, ws)
    else:
        fn = b2.b2_dgemm if a.dtype == "d" else b2.b2_sgemm

        def run():
            fn(a.transa, a.transb, a.m, a.n, a.k, a.alpha, A, lda, B, ldb, a.beta, C, ldc, variant=a.variant)

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
    print(json.dumps({"dtype": a.dtype, "trans": a.transa + a.transb, "m": a.m, "n": a.n, "k": a.k,
                      "variant": a.variant, "ms_per_launch": ms, "gflops": flops / ms / 1e6}))


if __name__ == "__main__":
    main()
