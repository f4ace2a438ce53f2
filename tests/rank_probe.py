"""Helper for test_sharding_gloo: one rank of a local launch.  Joins a gloo group from the launcher's
environment, takes its shard of a candidate range and reports through a MAX reduction; rank 0 prints
one JSON line."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch.distributed as dist  # noqa: E402

from paper_2201_13096_b200 import sharding  # noqa: E402


def main():
    n_total = int(sys.argv[1])
    assert sharding.under_launcher()
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    start, count = sharding.shard_range(n_total, rank, world)
    worst = sharding.max_over_ranks(float(rank + 1))
    counts = [None] * world
    dist.all_gather_object(counts, (start, count))
    if rank == 0:
        print(json.dumps({"n_gpus": world, "worst": worst, "shards": counts}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
