"""Worker of the two-rank CPU test: the replica bookkeeping of bench.py under gloo."""
import json
import os
import sys

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    dist.barrier()
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, device="cpu")
    out = {"rank": rank, "world": world, "ms": ms, "value": bench.job_value(world, 100, ms),
           "seed": bench.replica_seed(1, rank)}
    with open(os.path.join(sys.argv[1], "rank%d.json" % rank), "w") as f:
        json.dump(out, f)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
