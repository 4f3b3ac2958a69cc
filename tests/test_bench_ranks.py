"""bench.py with more than one rank: replicas only, no collective in the data path.  What the
ranks exchange is the timing (maximum over ranks) — checked here with two gloo ranks on CPU,
both through the helpers and through bench.py's own launcher of N ranks."""
import json
import os
import subprocess
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


def test_launcher_starts_n_ranks_and_the_blocks_are_the_slowest_ranks(capfd):
    """bench.launch_ranks (what `bench.py --gpus N` runs when no torchrun environment is set)
    with two CPU ranks and a stubbed step: both ranks time the same number of blocks, a block
    lasts as long as the slower rank's, and the job's throughput counts both ranks' units."""
    sys.path.insert(0, ROOT)
    import bench
    rc = bench.launch_ranks(2, os.path.join(ROOT, "tests", "rank_stub.py"), ["--steps", "3"], require_gpus=False,
                            timeout=300)
    assert rc == 0
    out = capfd.readouterr().out
    line = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["blocks"] >= 4
    (b0, c0), (b1, c1) = line["per_rank"]
    assert b0 == b1 == line["blocks"] and c0 == c1 == 3 * b0
    assert 1.9 <= line["ms_per_step"] < 6.0                 # rank 1's 2 ms per step, not rank 0's 1 ms
    assert abs(line["value"] - 2 * 10 / (line["ms_per_step"] * 1e-3)) < 1e-6 * line["value"]


def test_more_ranks_than_gpus_is_refused_loudly():
    """`bench.py --gpus 2` on a node with fewer than two CUDA devices must not run as N = 1."""
    import torch
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        import pytest
        pytest.skip("this node has two GPUs")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode != 0
    assert "refusing to run 2 ranks" in r.stderr and "{" not in r.stdout


def test_timed_blocks_stop_rule():
    sys.path.insert(0, ROOT)
    import bench
    n = [0]

    def block():
        n[0] += 1
        return 10.0
    ident = lambda v: v
    assert len(bench.timed_blocks(block, ident, min_blocks=20, min_total_ms=500.0)) == 50     # 0.5 s of 10 ms blocks
    assert len(bench.timed_blocks(lambda: 100.0, ident, min_blocks=20, min_total_ms=500.0)) == 20
    assert len(bench.timed_blocks(block, ident, exact_blocks=3)) == 3
    st = bench.block_stats([3.0, 1.0, 2.0], 2)
    assert st["ms_per_step"] == 1.0 and st["ms_per_step_min"] == 0.5 and st["blocks"] == 3
