"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own timing;
the reported time is the slowest rank's and the throughput counts every rank's
batch (the forward pass shards over the batch with no collective)."""
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
    local_ms = 10.0 + 5.0 * rank  # rank 1 is slower
    dist.barrier()
    slowest = bench.slowest_rank_ms(local_ms, world)
    value = bench.aggregate_images_per_s(world, 100, 4, slowest)
    out[rank] = (slowest, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_rank_and_the_whole_job():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slowest, value = res[0]
    assert slowest == 15.0
    assert abs(value - 2 * 100 * 4 / 15.0e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank_ms(7.5, 1) == 7.5
    assert bench.aggregate_images_per_s(1, 100, 20, 100.0) == 20000.0
