"""Worker of the world-size-2 CPU test: the rank plumbing bench.py uses under torchrun (gloo here)."""
import json
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank runs its own replica; the reported time is the slowest rank's
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")
    assert ms == 10.0 + 5.0 * (world - 1), ms
    # whole-job throughput counts the units of all ranks against that time
    tokens = 16 * world
    out = {"rank": rank, "ms": ms, "value": tokens / (ms * 1e-3)}
    dist.barrier()
    if rank == 0:
        print(json.dumps(out))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
