"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own timing;
the reported time is the slowest rank's and the throughput counts every rank's
batch (the forward pass shards over the batch with no collective).  The
training step's one exchange, the gradient all-reduce, is checked with the CPU
checker standing in for the device: the mean of the ranks' half-batch gradients
is the whole batch's gradient, and every rank takes the same SGD step."""
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


def _grad_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import numpy as np
    import bench
    import oracle
    from test_oracle_pins import TINY, tiny_inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    params, x, labels = tiny_inputs(N=4)
    half = slice(2 * rank, 2 * rank + 2)  # this rank's shard of the batch
    _, g, _ = oracle.backward(TINY, params, x[half], labels[half])
    t = torch.from_numpy(g.copy())
    bench.average_gradients(t, world)
    # the overlapped exchange of the training step averages the buffer in two buckets (the dense layers'
    # gradients first, the convolution layers' at the end of the pass): same result as one all-reduce
    t2 = torch.from_numpy(g.copy())
    cut = t2.numel() // 3
    bench.average_gradients(t2[cut:], world)
    bench.average_gradients(t2[:cut], world)
    assert torch.equal(t, t2)
    out[rank] = oracle.sgd_step(params, t2.numpy(), 0.1)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_average_to_the_whole_batch_gradient():
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import numpy as np
    import oracle
    from test_oracle_pins import TINY, tiny_inputs
    world = 2
    port = 31500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_grad_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    params, x, labels = tiny_inputs(N=4)
    _, g_all, _ = oracle.backward(TINY, params, x, labels)
    want = oracle.sgd_step(params, g_all, 0.1)
    assert np.array_equal(res[0], res[1])  # replicas stay identical
    assert np.allclose(res[0], want, rtol=1e-12, atol=1e-14)


def test_bench_gpus_n_starts_n_ranks_by_itself():
    """`python bench.py --gpus 2` with no launcher in the environment must start two ranks (here CPU ranks
    over gloo, plumbing only) and report the whole job: n_gpus 2, the slowest rank's time, both batches."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo", "--dry",
                        "--steps", "4"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2
    assert abs(out["ms_per_step"] - 11.0) < 1e-9          # rank 1 pretends 11 ms per step: the slowest rank's
    assert abs(out["value"] - 2 * 100 / 11e-3) < 1e-6    # both ranks' batches count
    assert abs(out["mean_gradient"] - 1.5) < 1e-12       # mean of the ranks' constant gradients 1 and 2
