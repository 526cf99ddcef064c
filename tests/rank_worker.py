"""A stand-in rank for the multi-rank plumbing test: joins the group the way bench.py's ranks do (environment
set by torch.distributed.run, gloo instead of NCCL), reports a canned time that differs per rank, and lets rank 0
print the result line.  Run by tests/test_sharding.py through shard.spawn_ranks; not a test itself."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2412_12706_b200 import shard  # noqa: E402


def main():
    dist, rank, world, local = shard.init_ranks("gloo")
    seconds = shard.max_over_ranks(0.5 * (rank + 1), dist)          # canned timings: rank r "took" 0.5 (r + 1) s
    mine = list(shard.rank_units(7, rank, world))
    everyone = [None] * world
    if dist is not None:
        dist.all_gather_object(everyone, mine)
    if rank == 0:
        line = shard.job_line("units_per_s", "1/s", 10.0, world, seconds, units=everyone)
        print(json.dumps(line), flush=True)
    shard.finish_ranks(dist)


if __name__ == "__main__":
    main()
