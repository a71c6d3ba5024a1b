"""Host-side logic of the multi-GPU benchmark: independent replicas, one problem per rank.

GEMM tiles are independent, so N GPUs run N independent problems with no data-path collective.
The only communication is a barrier and a max-reduction of the measured time, done through
``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of rank's replica: distinct problems on distinct ranks, rank 0 keeps the single-GPU seed."""
    return base_seed + 1000 * rank


def max_over_ranks(local_value: float, dist=None, device="cpu") -> float:
    """Largest ``local_value`` over all ranks (the time of the slowest rank); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_value)
    t = torch.tensor([local_value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gflops(flops_per_step: float, steps: int, local_ms: float, world: int, dist=None, device="cpu") -> tuple:
    """Whole-job GFLOP/s of `world` replicas that each ran `steps` steps: all flops over the slowest rank's time.

    Returns (gflops, ms) with ms the max over ranks."""
    ms = max_over_ranks(local_ms, dist, device)
    return world * flops_per_step * steps / (ms * 1e-3) / 1e9, ms
