"""Worker of test_bench_ranks_cpu.py: one gloo rank exercising bench.py's multi-rank plumbing on the CPU."""
import json
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    local_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
    dist.barrier()
    total = bench.rank_max(local_ms, world)
    out = {"rank": rank, "world": world, "seed": bench.shard_seed(rank), "total_ms": total,
           "tops": bench.job_tops(1e12, 5, world, total)}
    with open(os.path.join(sys.argv[1], "rank%d.json" % rank), "w") as f:
        json.dump(out, f)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
