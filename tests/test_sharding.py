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


def test_spawned_ranks_print_one_line_for_the_whole_job(capfd):
    """The spawn code bench.py uses for --gpus N (torch.distributed.run on 127.0.0.1) with two gloo ranks on CPU:
    rank 0's line reports both ranks, the slowest rank's time and disjoint units."""
    import json
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_worker.py")
    rc = shard.spawn_ranks(2, [worker], timeout=300)
    out = capfd.readouterr().out
    assert rc == 0
    lines = [json.loads(l) for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert line["value"] == 10.0 * 2 / 1.0                            # all ranks' units over the slowest rank's second
    assert sorted(line["units"][0] + line["units"][1]) == list(range(7))
