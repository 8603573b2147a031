"""Data-parallel sharding of the path: segments / sequences are independent, so ranks split
them and never exchange payload.  Only timing is reduced across ranks."""

from __future__ import annotations

from typing import Tuple


def shard_range(n_units: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) of `n_units` independent units owned by `rank`: sizes differ by
    at most one, earlier ranks take the larger shards, every unit has exactly one owner."""
    if world < 1 or not 0 <= rank < world or n_units < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput_gbs(bytes_per_rank: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job GB/s when every rank moves `bytes_per_rank` per step (weak scaling) and the
    slowest rank needs `ms_per_step_max`."""
    return world * bytes_per_rank / (ms_per_step_max * 1e-3) / 1e9
