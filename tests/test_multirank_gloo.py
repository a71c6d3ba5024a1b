"""The N > 1 benchmark path on CPU: two gloo ranks, independent replicas, max-over-ranks timing."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1611_08035_b200 import replicas, synth


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 if rank == 0 else 25.0  # rank 1 is the slow one
        gflops, ms = replicas.aggregate_gflops(2.0e9, 4, local_ms, world, dist)
        seed = replicas.rank_seed(2013, rank)
        A = synth.matrix(8, 8, 8, "uniform", seed)
        gathered = [torch.zeros_like(A) for _ in range(world)]
        dist.all_gather(gathered, A)
        out.put((rank, gflops, ms, seed, bool(torch.equal(gathered[0], gathered[1]))))
    finally:
        dist.destroy_process_group()


def test_two_rank_replicas_aggregate_on_the_slowest_rank():
    world, port = 2, 29517 + os.getpid() % 1000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, gflops, ms, seed, same in results:
        assert ms == 25.0  # every rank sees the max
        assert abs(gflops - world * 2.0e9 * 4 / 25.0e-3 / 1e9) < 1e-9
        assert seed == 2013 + 1000 * rank
        assert not same  # the replicas are different problems
    assert results[0][3] == 2013  # rank 0 keeps the single-GPU seed


def test_single_process_is_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    g, ms = replicas.aggregate_gflops(1e9, 2, 4.0, 1)
    assert ms == 4.0 and abs(g - 1e9 * 2 / 4e-3 / 1e9) < 1e-12
