"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own (fake) timings,
combine them exactly as bench.py does under torchrun -- the slowest rank sets the time, the job's
throughput is the sum of what all ranks processed.  MX blocks are independent, so the path has no
data exchange to test: ranks work on their own shards."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r is slower by r milliseconds in every phase
    local = [1.0 + rank, 0.5 + rank, 0.25 + rank, 0.125 + rank]
    got = bench.max_over_ranks(local, "cpu", world)
    units = 1000.0  # per rank
    thr = bench.job_throughput(units, world, got[1] * 1e-3)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(repr((got, thr)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_with_gloo(tmp_path):
    world = 2
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    results = [eval(open(tmp_path / f"r{r}.txt").read()) for r in range(world)]
    for got, thr in results:  # every rank sees the maximum over ranks
        assert got == [2.0, 1.5, 1.25, 1.125]
        assert thr == 2 * 1000.0 / 1.5e-3
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], "cpu", 1) == [3.0, 4.0]
    assert bench.job_throughput(10.0, 1, 2.0) == 5.0
