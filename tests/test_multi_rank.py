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


def test_clock_record_keeps_the_samples_inside_the_timed_region():
    """bench.py's clock record: nvidia-smi lines carry timestamps, and only those between the two
    host times that bracket the timed region count; throttle reasons are collected from them."""
    import datetime
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench

    base = datetime.datetime(2026, 1, 2, 3, 4, 5)

    def line(ms, sm, power, cap="Not Active", hw="Not Active"):
        t = (base + datetime.timedelta(milliseconds=ms)).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
        return f"{t}, {sm}, 1965, {power}, {hw}, Not Active, Not Active, {cap}"

    text = "\n".join([line(0, 345, 150.0), line(10, 1965, 300.0), line(20, 1905, 420.0, cap="Active"),
                      line(30, 1965, 310.0), line(500, 345, 140.0, hw="Active"), "garbage line"])
    t0 = (base + datetime.timedelta(milliseconds=5)).timestamp()
    t1 = (base + datetime.timedelta(milliseconds=35)).timestamp()
    rec = bench.ClockSampler.summarize(text, t0, t1)
    assert rec["in_timed_region"] and rec["samples"] == 3
    assert rec["sm_mhz"] == 1965 and rec["sm_max_mhz"] == 1965 and rec["power_w_max"] == 420.0
    assert rec["reasons"] == ["sw_power_cap"]  # the hw_slowdown sample lies outside the region
    # a region that caught no sample: the samples taken under load stand in, and the record says so
    rec = bench.ClockSampler.summarize(text, t1 + 100, t1 + 101)
    assert not rec["in_timed_region"] and rec["samples"] == 3
    assert bench.ClockSampler.summarize("", t0, t1)["reasons"] == ["no samples"]
