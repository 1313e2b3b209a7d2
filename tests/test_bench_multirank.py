"""The multi-rank arithmetic of bench.py on CPU: two gloo ranks, max-over-ranks time, aggregate rate.

The attention path shards by sequence / kv head with no collective on the data path, so the only
cross-rank step of the benchmark is the reduction of the per-rank times; this checks it with
world_size 2 without a GPU.
"""
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
    ms_local = 10.0 + 5.0 * rank                   # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, torch.device("cpu"))
    out[rank] = (ms, bench.whole_job_rate(16, 100, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_rate():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        ms, rate = res[rank]
        assert ms == 15.0                          # max over ranks, known to every rank
        assert abs(rate - 2 * 16 * 100 / 15e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.whole_job_rate(16, 10, 1, 2.0) == 16 * 10 / 2e-3
