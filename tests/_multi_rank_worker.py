"""Worker of tests/test_bench_multi.py: one gloo rank exercising bench.py's multi-rank helpers."""
import json
import os
import sys
from pathlib import Path

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))

import torch
import torch.distributed as dist

import bench


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    device = torch.device("cpu")
    # every rank times its own replica; the job's time is the slowest rank's
    mine = 10.0 + 5.0 * rank
    slowest = bench.max_over_ranks(mine, dist, device)
    value = bench.whole_job_value(world, 24, 7, slowest * 1e-3)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"slowest": slowest, "value": value, "world": world}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
