"""The N>1 host logic on CPU: two gloo ranks agree on disjoint units and on the max time."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_12706_b200 import shard


def test_rank_units_partition():
    for n in (0, 1, 7, 8, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                u = shard.rank_units(n, r, world)
                seen += list(u)
                assert abs(len(u) - n / world) < 1
            assert seen == list(range(n))
    seeds = {shard.sequence_seed(5, r, 4, s) for r in range(8) for s in range(4)}
    assert len(seeds) == 32


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = list(shard.rank_units(5, rank, world))
    t = shard.max_over_ranks(1.0 + rank, dist)          # rank 1 is the slow one
    gathered = [None] * world
    dist.all_gather_object(gathered, units)
    q.put((rank, t, gathered))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, t, gathered in res:
        assert t == 2.0                                   # max over ranks
        assert sorted(gathered[0] + gathered[1]) == list(range(5))
        assert not set(gathered[0]) & set(gathered[1])
    assert shard.whole_job_throughput(10.0, 2, 2.0) == 10.0
