"""Worker of tests/test_multirank_cpu.py: one rank of a CPU (gloo) job that exercises the part of
bench.py's multi-rank path that needs no GPU: the MAX-over-ranks timing and the whole-job throughput."""
import json
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    # rank k "measured" 10 (k + 1) ms for 4 steps of 1000 elements
    ms, value = bench.whole_job_throughput(10.0 * (rank + 1), 1000, 4, world, torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms_total": ms, "value": value, "world": world}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
