"""Worker of tests/test_multi_rank_cpu.py: one rank of a CPU (gloo) run of the benchmark's
multi-rank plumbing -- rendezvous, barrier, max-over-ranks timing and whole-job aggregation.
Rank 0 prints one JSON line."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def main():
    rank, world, local = bench.dist_setup(int(os.environ.get("WORLD_SIZE", "1")))
    bench.barrier(world)
    # every rank "measures" a different step time; the job's time is the slowest rank's
    ms = bench.max_over_ranks(10.0 * (rank + 1), world)
    tokens_per_rank, steps = 1000, 4
    value = bench.aggregate(tokens_per_rank, world, ms, steps)
    bench.barrier(world)
    if rank == 0:
        print(json.dumps({"world": world, "local": local, "ms": ms, "value": value}), flush=True)
    import torch.distributed as dist
    if dist.is_initialized():
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
