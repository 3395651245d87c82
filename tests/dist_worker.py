"""One rank of the two-process CPU check of the benchmark's multi-rank arithmetic (gloo).

Launched by test_bench_launch.py under torch.distributed.run; rank 0 prints one JSON line.
"""
import json
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # every rank "measured" a different time; the job's time is the slowest rank's
    mine = 10.0 + 5.0 * rank
    total = bench.max_over_ranks(mine, world, device="cpu")
    value = bench.whole_job_value(1000, 4, world, total)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"world": world, "total_ms": total, "value": value}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
