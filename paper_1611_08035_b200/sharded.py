"""GEMM over several GPUs with distributed operands: all-gather of A's panels into local memory, local kernel.

C tiles are independent, so C (and B) are split by column panels: rank r owns the columns
``col_range(n, W, r)`` of B (k x n_r) and of C (m x n_r).  A (m x k) is distributed too, by k-panels: rank q
holds the columns ``col_range(k, W, q)`` of A.  Every rank needs all of A, so the one exchange step is an
all-gather of A's panels (NCCL over NVLink on GPUs).  The gathered panels land in this GPU's own memory and
the unchanged single-GPU kernel reads them from there; nothing reads a peer's memory directly.

To overlap the exchange with arithmetic, each rank's panel is cut into ``sub_panels`` slices.  Slice s of
every rank is gathered on a communication stream while the compute stream multiplies slice s-1:

    for s in slices:   gather slice s of all W panels          (communication stream)
    for s in slices:   for q in ranks:                          (compute stream, after slice s arrived)
                           C_r := alpha * A_q[:, slice s] * B_r[rows of that slice, :] + beta' * C_r

with beta' = beta for the first product and 1 afterwards.  The order of the partial products is fixed by
(W, sub_panels), so results are reproducible; on integer-valued data they equal the single-GPU result bit
for bit, otherwise they satisfy the same 2*k*u*S bound (a different but fixed summation order).

The same schedule runs on CPU tensors with the gloo backend when a ``gemm`` callable is passed in (the tests
do that); without one the CUDA library is used and CPU tensors are rejected.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch


def col_range(total: int, world: int, rank: int) -> tuple:
    """Contiguous balanced split: the first ``total % world`` ranks get one extra column."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def panel_width(total: int, world: int) -> int:
    """Width every rank's panel buffer is padded to (the widest panel), at least 1."""
    return max(1, -(-total // world))


def slices(width: int, sub_panels: int) -> list:
    """Cut [0, width) into at most ``sub_panels`` contiguous slices of equal width (the last may be shorter)."""
    sub_panels = max(1, min(sub_panels, width))
    step = -(-width // sub_panels)
    return [(lo, min(width, lo + step)) for lo in range(0, width, step)]


def _device_gemm(dtype) -> Callable:
    from . import binding  # fails loudly when the CUDA library is missing

    if dtype == torch.float64:
        return binding.b2_dgemm
    if dtype == torch.float32:
        return binding.b2_sgemm
    raise TypeError("sharded_gemm takes float64 or float32 operands")


def local_products(m: int, n: int, k: int, alpha: float, gathered: torch.Tensor, B_cols: torch.Tensor, beta: float,
                   C_cols: torch.Tensor, world: int, rank: int, cuts: list, gemm: Callable, wait=None) -> None:
    """The compute half of ``sharded_gemm`` for rank ``rank`` of ``world``: one GEMM per (slice, source rank).

    ``gathered`` holds, for slice (lo, hi) of ``cuts``, the W slices of width hi-lo back to back starting at
    element W*m*lo (rank q's at W*m*lo + q*m*(hi-lo)).  ``wait(s)`` is called before slice s is used.
    """
    n0, n1 = col_range(n, world, rank)
    nr = n1 - n0
    first = True
    for s, (lo, hi) in enumerate(cuts):
        if wait is not None:
            wait(s)
        width = hi - lo
        for q in range(world):
            k0, k1 = col_range(k, world, q)
            valid = min(hi, k1 - k0) - lo  # columns of this slice that exist in rank q's panel
            if valid <= 0 or nr == 0:
                continue
            a = gathered[world * m * lo + q * m * width:]
            b = B_cols[k0 + lo:]
            gemm("N", "N", m, nr, valid, alpha, a, max(1, m), b, max(1, k), beta if first else 1.0, C_cols, max(1, m))
            first = False
    if first and nr > 0:  # k == 0: C := beta*C
        gemm("N", "N", m, nr, 0, alpha, gathered, max(1, m), B_cols, max(1, k), beta, C_cols, max(1, m))


def sharded_gemm(m: int, n: int, k: int, alpha: float, A_panel: torch.Tensor, B_cols: torch.Tensor, beta: float,
                 C_cols: torch.Tensor, group=None, sub_panels: int = 4, gemm: Optional[Callable] = None,
                 gathered: Optional[torch.Tensor] = None) -> torch.Tensor:
    """C := alpha*A*B + beta*C (no transposes) with A, B and C distributed over the ranks of ``group``.

    Per rank (W ranks, this one is r; all storage column-major and flat):
      A_panel  m x panel_width(k, W), ld = m: columns col_range(k, W, r) of A, padding columns ignored
      B_cols   k x n_r, ld = k:               columns col_range(n, W, r) of B
      C_cols   m x n_r, ld = m:               the same columns of C, updated in place
      gathered optional scratch of W * m * panel_width(k, W) elements (allocated when absent)

    Returns C_cols.  Collective: every rank of the group must call it with the same m, n, k and sub_panels.
    """
    import torch.distributed as dist

    grouped = dist.is_initialized()
    world = dist.get_world_size(group) if grouped else 1
    rank = dist.get_rank(group) if grouped else 0
    kw = panel_width(k, world)
    n0, n1 = col_range(n, world, rank)
    nr = n1 - n0
    on_gpu = A_panel.is_cuda
    if gemm is None:
        if not on_gpu:
            raise RuntimeError("sharded_gemm without a gemm callable runs the CUDA library: operands must be CUDA tensors")
        gemm = _device_gemm(A_panel.dtype)
    if A_panel.numel() < m * kw or B_cols.numel() < k * nr or C_cols.numel() < m * nr:
        raise ValueError("operand storage smaller than its shape")
    if gathered is None:
        gathered = torch.empty(world * max(1, m) * kw, dtype=A_panel.dtype, device=A_panel.device)
    elif gathered.numel() < world * m * kw:
        raise ValueError("gathered scratch too small")
    if m == 0:
        return C_cols

    cuts = slices(kw, sub_panels)
    # ---- exchange: slice s of every rank's panel -> gathered[W*m*lo : W*m*hi] viewed as (W, m*(hi-lo)) ----
    arrived = []
    if on_gpu:
        compute = torch.cuda.current_stream()
        comm = _comm_stream(A_panel.device)
        comm.wait_stream(compute)  # the panels and the scratch are ready when the compute stream gets here
    for lo, hi in cuts:
        src = A_panel[m * lo: m * hi]
        dst = gathered[world * m * lo: world * m * hi]
        if not grouped:  # no process group: a single rank, the exchange is a copy
            ctx = torch.cuda.stream(comm) if on_gpu else _NullCtx()
            with ctx:
                dst.copy_(src)
        elif on_gpu:
            with torch.cuda.stream(comm):
                dist.all_gather_into_tensor(dst, src.contiguous(), group=group)
        else:
            parts = [dst[q * m * (hi - lo): (q + 1) * m * (hi - lo)] for q in range(world)]
            dist.all_gather(parts, src.contiguous(), group=group)
        if on_gpu:
            ev = torch.cuda.Event()
            ev.record(comm)
            arrived.append(ev)

    local_products(m, n, k, alpha, gathered, B_cols, beta, C_cols, world, rank, cuts, gemm,
                   wait=(lambda s: compute.wait_event(arrived[s])) if on_gpu else None)
    if on_gpu:
        gathered.record_stream(comm)
    return C_cols


class _NullCtx:
    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


_COMM_STREAMS: dict = {}


def _comm_stream(device) -> "torch.cuda.Stream":
    key = torch.device(device).index if torch.device(device).index is not None else torch.cuda.current_device()
    if key not in _COMM_STREAMS:
        _COMM_STREAMS[key] = torch.cuda.Stream(device=key)
    return _COMM_STREAMS[key]


def scatter_problem(m: int, n: int, k: int, A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, world: int, rank: int):
    """Cut full column-major A (ld m), B (ld k), C (ld m) into rank's shares (for tests and the demo runner)."""
    kw = panel_width(k, world)
    k0, k1 = col_range(k, world, rank)
    n0, n1 = col_range(n, world, rank)
    A_panel = torch.zeros(max(1, m) * kw, dtype=A.dtype, device=A.device)
    A_panel[: m * (k1 - k0)] = A[m * k0: m * k1]
    return A_panel, B[k * n0: k * n1].clone(), C[m * n0: m * n1].clone()


def main() -> None:
    """Timing run under torchrun (one rank per GPU, NCCL): ``torchrun --nproc-per-node N -m paper_1611_08035_b200.sharded``."""
    import argparse
    import json
    import os

    import torch.distributed as dist

    from . import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("-m", type=int, default=8192)
    ap.add_argument("-n", type=int, default=8192)
    ap.add_argument("-k", type=int, default=8192)
    ap.add_argument("--sub-panels", type=int, default=4)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    rank, world = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    dist.init_process_group("nccl", rank=rank, world_size=world)
    try:
        m, n, k = args.m, args.n, args.k
        k0, k1 = col_range(k, world, rank)
        n0, n1 = col_range(n, world, rank)
        kw = panel_width(k, world)
        # every rank draws only its own share: element (r, c) of the full matrix is a function of (seed, index)
        A_panel = torch.zeros(m * kw, dtype=torch.float64, device="cuda")
        A_panel[: m * (k1 - k0)] = synth.matrix(m, k, m, "uniform", 11, device="cuda")[m * k0: m * k1]
        B_cols = synth.matrix(k, n, k, "uniform", 112, device="cuda")[k * n0: k * n1].clone()
        C_cols = synth.matrix(m, n, m, "uniform", 213, device="cuda")[m * n0: m * n1].clone()
        scratch = torch.empty(world * m * kw, dtype=torch.float64, device="cuda")
        for _ in range(args.warmup):
            sharded_gemm(m, n, k, 1.5, A_panel, B_cols, 0.5, C_cols, sub_panels=args.sub_panels, gathered=scratch)
        torch.cuda.synchronize()
        dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.iters):
            sharded_gemm(m, n, k, 1.5, A_panel, B_cols, 0.5, C_cols, sub_panels=args.sub_panels, gathered=scratch)
        e1.record()
        torch.cuda.synchronize()
        t = torch.tensor([e0.elapsed_time(e1) / args.iters], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        if rank == 0:
            ms = float(t.item())
            print(json.dumps({"workload": f"sharded_dgemm_nn_{m}x{n}x{k}", "n_gpus": world, "ms": ms,
                              "gflops": 2.0 * m * n * k / (ms * 1e-3) / 1e9, "sub_panels": args.sub_panels}))
    finally:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
