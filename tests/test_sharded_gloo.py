"""The distributed-operand GEMM schedule on CPU: gloo ranks, the oracle as the local GEMM.

What is checked is the host logic of the multi-GPU path: the partition of A, B and C, the all-gather of the
slices of A's panels into local scratch, which slice of which rank's panel meets which rows of B, and the
beta handling across the partial products.  Integer-valued data must reproduce the oracle's full GEMM bit for
bit; uniform data must stay within the 2*k*u*S bound."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1611_08035_b200 import sharded, synth


def _oracle_gemm():
    import sys
    from pathlib import Path

    root = str(Path(__file__).resolve().parent.parent)
    if root not in sys.path:
        sys.path.insert(0, root)
    from oracle import ref as oracle

    oracle.lib()

    def gemm(ta, tb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc):
        oracle.ref_gemm(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, C.numpy(), ldc)
        return 0

    return oracle, gemm


CASES = [(37, 29, 23, 3, "int9"), (64, 50, 41, 4, "uniform"), (5, 3, 1, 2, "int9"), (16, 7, 0, 2, "int9"),
         (33, 1, 9, 8, "uniform")]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        oracle, gemm = _oracle_gemm()
        verdicts = []
        for (m, n, k, sub, dist_name) in CASES:
            A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, dist_name, 7000 + m)
            A_panel, B_cols, C_cols = sharded.scatter_problem(m, n, k, A, B, C, world, rank)
            sharded.sharded_gemm(m, n, k, 1.5, A_panel, B_cols, 0.5, C_cols, sub_panels=sub, gemm=gemm)
            want = C.numpy().copy()
            oracle.ref_gemm("N", "N", m, n, k, 1.5, A.numpy(), lda, B.numpy(), ldb, 0.5, want, ldc)
            _, S = oracle.ref_gemm_hi("N", "N", m, n, k, 1.5, A.numpy(), lda, B.numpy(), ldb, 0.5, C.numpy(), ldc)
            n0, n1 = sharded.col_range(n, world, rank)
            mine, got = want[m * n0: m * n1], C_cols.numpy()
            if dist_name == "int9":
                verdicts.append(mine.tobytes() == got.tobytes())
            else:
                bound = 2.0 * max(k, 1) * 2.0 ** -53 * S[m * n0: m * n1]
                verdicts.append(bool(np.all(np.abs(mine - got) <= bound)))
        out.put((rank, verdicts))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_gemm_matches_the_oracle_on_every_rank(world):
    port = 29600 + os.getpid() % 300 + world
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, verdicts in results:
        assert all(verdicts), f"rank {rank}: {verdicts}"


def test_partition_helpers():
    for total in (0, 1, 7, 64, 1001):
        for world in (1, 2, 3, 8):
            ranges = [sharded.col_range(total, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            widths = [hi - lo for lo, hi in ranges]
            assert max(widths) - min(widths) <= 1 and max(widths) <= sharded.panel_width(total, world)
    assert sharded.slices(10, 4) == [(0, 3), (3, 6), (6, 9), (9, 10)]
    assert sharded.slices(2, 4) == [(0, 1), (1, 2)]
    assert sharded.slices(1, 1) == [(0, 1)]


def test_cpu_tensors_need_an_explicit_gemm():
    A = torch.zeros(4, dtype=torch.float64)
    with pytest.raises(RuntimeError):
        sharded.sharded_gemm(2, 2, 2, 1.0, A, A, 0.0, A.clone())
