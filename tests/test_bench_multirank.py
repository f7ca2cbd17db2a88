"""Host-side logic of `bench.py --gpus N` on CPU with two gloo ranks: ranks draw different token
batches, the job's time is the maximum over ranks, and the aggregate counts every rank's work.
(The GPU path itself shards over token batches with no data-path collective.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
        red = bench.max_over_ranks(ms, dist, device="cpu")
        seeds = [bench.rank_seed(rank, i) for i in range(bench.N_SETS)]
        gathered = [None] * world
        dist.all_gather_object(gathered, seeds)
        out.put((rank, red, gathered))
    finally:
        dist.destroy_process_group()


def test_two_rank_reduction_and_seeds():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, gathered in res:
        assert red == [15.0, 3.0]                        # maximum over ranks, element-wise
        flat = [s for seeds in gathered for s in seeds]
        assert len(set(flat)) == len(flat)               # no two (rank, set) pairs share a batch


def test_single_process_is_identity_and_aggregate_is_linear_in_ranks():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    one = bench.aggregate_tops(1, 2e11, 10, 5.0)
    assert abs(one - 2e11 * 10 / 5e-3 / 1e12) < 1e-9
    assert abs(bench.aggregate_tops(8, 2e11, 10, 5.0) - 8 * one) < 1e-9
