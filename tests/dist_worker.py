"""Worker of the world_size-2 CPU test of the bench's multi-rank logic (gloo backend).

Launched by tests/test_bench_ranks.py through torch.distributed.run; every rank contributes its own
fake durations, rank 0 writes what the bench's helpers make of them."""
import json
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    out = sys.argv[1]
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    step_ms, e2e_ms = (10.0, 30.0) if rank == 0 else (12.5, 20.0)      # each rank is the slower one once
    dist.barrier()
    worst = bench.slowest_rank([step_ms, e2e_ms], world, "cpu")
    if rank == 0:
        with open(out, "w") as f:
            json.dump(dict(world=world, worst=worst, value=bench.job_value(world, 1, 61, worst[0]),
                           seeds=[bench.request_seed(0, r) for r in range(world)]), f)
    # the reference arm runs on rank 0 alone: the other ranks return without touching the oracle
    if rank != 0:
        assert bench.run_reference(None, None) is None
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
