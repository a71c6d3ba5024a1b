"""The distributed-operand GEMM on one GPU: the exchange through NCCL with a single rank, and the compute half
for every rank of a 4-rank job run one after another over hand-assembled gathered panels (one process, no rank
waits on another)."""
import os

import numpy as np
import pytest
import torch

from gpu_util import sample_columns
from paper_1611_08035_b200 import sharded, synth

pytestmark = pytest.mark.gpu


def test_single_rank_nccl_exchange_and_overlap_streams(b2, oracle):
    import torch.distributed as dist

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(29700 + os.getpid() % 200)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        m, n, k = 1024, 768, 520
        for dist_name, exact in (("int9", True), ("uniform", False)):
            A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, dist_name, 8100)
            A_panel, B_cols, C_cols = (t.cuda() for t in sharded.scatter_problem(m, n, k, A, B, C, 1, 0))
            for _ in range(2):  # the second call reuses the scratch the first one is still reading
                Cd = C_cols.clone()
                scratch = torch.empty(m * k, dtype=torch.float64, device="cuda")
                sharded.sharded_gemm(m, n, k, 1.5, A_panel, B_cols, 0.5, Cd, sub_panels=5, gathered=scratch)
            assert b2.b2_device_status() == 0
            want = C.numpy().copy()
            oracle.ref_gemm("N", "N", m, n, k, 1.5, A.numpy(), lda, B.numpy(), ldb, 0.5, want, ldc)
            got = Cd.cpu().numpy()
            if exact:
                assert got.tobytes() == want.tobytes()
            else:
                _, S = oracle.ref_gemm_hi("N", "N", m, n, k, 1.5, A.numpy(), lda, B.numpy(), ldb, 0.5, C.numpy(), ldc)
                assert np.all(np.abs(got - want) <= 2.0 * k * 2.0 ** -53 * S)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [4, 3])
def test_every_rank_of_a_job_computed_in_turn(b2, oracle, world):
    m, n, k, sub = 1000, 1030, 777, 3
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 8200 + world)
    shares = [sharded.scatter_problem(m, n, k, A, B, C, world, r) for r in range(world)]
    kw = sharded.panel_width(k, world)
    cuts = sharded.slices(kw, sub)
    gathered = torch.empty(world * m * kw, dtype=torch.float64)
    for lo, hi in cuts:  # what the all-gather of slice (lo, hi) leaves in the scratch
        for q in range(world):
            gathered[world * m * lo + q * m * (hi - lo): world * m * lo + (q + 1) * m * (hi - lo)] = \
                shares[q][0][m * lo: m * hi]
    gathered = gathered.cuda()
    want = C.numpy().copy()
    oracle.ref_gemm("N", "N", m, n, k, -1.0, A.numpy(), lda, B.numpy(), ldb, 1.0, want, ldc)
    for r in range(world):
        n0, n1 = sharded.col_range(n, world, r)
        Cd = shares[r][2].cuda()
        sharded.local_products(m, n, k, -1.0, gathered, shares[r][1].cuda(), 1.0, Cd, world, r, cuts, b2.b2_dgemm)
        assert b2.b2_device_status() == 0
        assert Cd.cpu().numpy().tobytes() == want[m * n0: m * n1].tobytes(), f"rank {r}"
