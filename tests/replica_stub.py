"""Stand-in for bench.py in the launcher test: every replica joins a gloo group, applies the
benchmark's timing rule to a made-up per-rank time and rank 0 prints the result."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import torch.distributed as dist  # noqa: E402

import bench  # noqa: E402

if __name__ == "__main__":
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = bench.max_over_ranks(2.0 + rank)
    if rank == 0:
        with open(sys.argv[1], "w") as f:
            json.dump(dict(world=world, ms=ms, value=bench.aggregate_tokens_per_s(100, world, ms),
                           args=sys.argv[2:]), f)
    dist.destroy_process_group()
