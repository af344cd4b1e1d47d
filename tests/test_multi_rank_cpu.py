"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, the step time
is the max over ranks and the value the aggregate over replicas.  (The path has
no exchange step, so this reduction of timings is the only collective.)"""
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
        mine = [1.0 + rank, 5.0 - rank, 2.0]
        red = bench.reduce_max_over_ranks(mine)
        out[rank] = (red, bench.aggregate_throughput(10.0, world, red[0]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_aggregate():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(world):
        red, value = out[r]
        assert red == [2.0, 5.0, 2.0]
        assert value == 2 * 10.0 / 2.0


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert bench.aggregate_throughput(4.0, 1, 2.0) == 2.0
    ab = bench.algorithmic_bytes()
    assert ab["nt2"] == 4 * 64 * (1 << 24) and ab["os2"] == (2 * 8 + 16) * 124_439_808
    assert ab["os5"] == (2 * 4 + 16) * 1_300_000_000 and ab["acc5"] == 8 * (4 * 32 + 8) * (1 << 22)
    flops, launches = bench.model_flops()
    assert launches == 4 and flops == 4 * 12 * 2 * 32 * 1024 * (768 * 2304 + 768 * 768 + 2 * 768 * 3072)


def test_shard_bounds_partition_the_vector():
    from paper_2508_18182_b200.binding import shard_bounds
    for P in (0, 1, 7, 8, 9, 1000, 124_439_808, 1_300_000_000, 12345677):
        for world in (1, 2, 3, 4, 8, 13):
            prev = 0
            for r in range(world):
                lo, hi = shard_bounds(P, r, world)
                assert lo == prev and hi >= lo and (lo % 8 == 0 or lo == P)
                prev = hi
            assert prev == P
            sizes = [shard_bounds(P, r, world)[1] - shard_bounds(P, r, world)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 8 + 7        # balanced to within one aligned unit
