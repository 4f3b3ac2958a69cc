"""bench.py with more than one rank: replicas only, no collective in the data path.  What the
ranks exchange is the timing (maximum over ranks) — checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, ms_e2e = bench.max_over_ranks([10.0 + rank, 7.0 - rank], "cpu", world)   # rank 1 slower on the first
    value = bench.job_throughput(1024, 100, ms, world)
    out[rank] = (ms, ms_e2e, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_ranks_time_and_the_whole_jobs_units():
    world, port = 2, 29511 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, ms_e2e, value = res[0]
    assert ms == 11.0 and ms_e2e == 7.0
    assert abs(value - 2 * 1024 * 100 / 11e-3) < 1e-6 * value


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 2.0], "cpu", 1) == [3.5, 2.0]
    assert bench.job_throughput(8, 10, 2.0, 1) == 8 * 10 / 2e-3
