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


def init_ranks(backend: str = "nccl"):
    """Reads RANK / WORLD_SIZE / LOCAL_RANK / MASTER_* from the environment (as torch.distributed.run sets them) and
    joins the process group when there is more than one rank.  Returns (dist or None, rank, world, local_rank).
    The group exists only for the barrier and the max over ranks of the timings: the data path has no collective."""
    import os
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return None, rank, world, local
    import torch
    import torch.distributed as dist
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend)
    return dist, rank, world, local


def finish_ranks(dist) -> None:
    if dist is not None and dist.is_initialized():
        dist.destroy_process_group()


def spawn_ranks(n_ranks: int, script_and_args: list[str], port: int | None = None, timeout: float | None = None) -> int:
    """Starts `n_ranks` local processes of `script_and_args` under torch.distributed.run (one per GPU for the
    benchmark), rendezvous on 127.0.0.1, and returns the launcher's exit code.  The ranks inherit stdout, so
    rank 0's result line appears on the caller's."""
    import socket
    import subprocess
    import sys
    if port is None:
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + list(script_and_args)
    return subprocess.run(cmd, timeout=timeout).returncode


def job_line(metric: str, unit: str, units_per_rank: float, world: int, slowest_seconds: float, **more) -> dict:
    """The fields of a result line that depend on the number of ranks."""
    line = {"metric": metric, "value": whole_job_throughput(units_per_rank, world, slowest_seconds), "unit": unit,
            "n_gpus": world, "scaling": "weak"}
    line.update(more)
    return line
