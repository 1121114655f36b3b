"""Worker for the two-rank CPU test of the benchmark's aggregation (gloo backend)."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch.distributed as dist  # noqa: E402

import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    local_ms = 10.0 + 5.0 * rank                 # rank 1 is the slow one
    dist.barrier()
    worst = bench.max_over_ranks(local_ms)
    value = bench.replica_throughput(2.0e12, world, worst)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"world": world, "worst_ms": worst, "value": value}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
