"""Host-side sharding of the path over GPUs.

Every (sequence, layer, KV head) is an independent unit of the path: scoring, selection,
quantization groups and the decode softmax never cross KV heads, so ranks need no data-path
collective.  Ranks only agree on who owns which units and on the slowest rank's time.
"""
from __future__ import annotations


def rank_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous block partition of ``n_units`` independent units; sizes differ by at most one."""
    if not (0 <= rank < world) or n_units < 0:
        raise ValueError("bad rank/world/n_units")
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def sequence_seed(base_seed: int, rank: int, seqs_per_rank: int, s: int) -> int:
    """Seed of local sequence ``s`` on ``rank``: distinct for every (rank, s)."""
    return base_seed + 1000 * (rank * seqs_per_rank + s)


def max_over_ranks(x: float, dist=None, device=None) -> float:
    """Slowest rank's value (multi-GPU timings are the max over ranks)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: float, world: int, slowest_seconds: float) -> float:
    """Aggregate throughput of a weak-scaled job: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / slowest_seconds
