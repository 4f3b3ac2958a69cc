"""Stand-in for bench.py's GPU arm in the launcher test: started by bench.launch_ranks as one of
N CPU ranks (gloo), it times blocks of a stubbed step function with bench.timed_blocks and the
ranks' maximum, and rank 0 prints one JSON line.  No CUDA, no part of the method."""
import json
import os
import sys
import time

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def main():
    steps = int(sys.argv[sys.argv.index("--steps") + 1])
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    calls = [0]

    def step():                                   # the stub: rank r takes (1 + r) ms per step
        calls[0] += 1
        time.sleep(1e-3 * (1 + rank))

    def time_block():
        dist.barrier()
        t0 = time.perf_counter()
        for _ in range(steps):
            step()
        ms = 1e3 * (time.perf_counter() - t0)
        dist.barrier()
        return ms

    times = bench.timed_blocks(time_block, lambda v: bench.max_over_ranks(v, "cpu", world),
                               min_blocks=4, min_total_ms=30.0)
    st = bench.block_stats(times, steps)
    counts = [None] * world
    dist.all_gather_object(counts, (len(times), calls[0]))
    if rank == 0:
        print(json.dumps({"n_gpus": world, "blocks": st["blocks"], "ms_per_step": st["ms_per_step"],
                          "per_rank": counts, "value": bench.job_throughput(10, 1, st["ms_per_step"], world)}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
