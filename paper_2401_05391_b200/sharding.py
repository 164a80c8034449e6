"""Host-side logic for running the path on several GPUs (one process per GPU).

The path has no exchange step: every (request, kv head) work group is an
independent problem.  So ranks either hold their own requests (what
``bench.py --gpus N`` does: weak scaling, per-rank work fixed) or a slice of
the kv heads of the same requests (how the paper spreads a layer over tiles
with tensor parallelism, Section 4); the tiny beam-parent table is replicated
and nothing is communicated on the data path.  Only timing crosses ranks.
"""
from __future__ import annotations

from typing import Optional

import torch

from .workloads import Workload


def rank_workload(w: Workload, rank: int, world: int) -> Workload:
    """The workload rank ``rank`` runs under weak scaling: same shape, its own
    requests (a distinct seed family per rank)."""
    if not 0 <= rank < world:
        raise ValueError("rank outside [0, world)")
    return w if world == 1 else w.scaled(index=w.index + 100 * rank)


def shard_heads(w: Workload, rank: int, world: int):
    """Head-sharded view for rank ``rank``: (workload with heads/world heads,
    slice of query heads, slice of kv heads).  kv_heads must divide evenly."""
    if w.kv_heads % world or w.heads % world:
        raise ValueError("heads and kv_heads must be multiples of the world size")
    hq, hk = w.heads // world, w.kv_heads // world
    sub = w.scaled(heads=hq, kv_heads=hk, name=f"{w.name}[tp{rank}/{world}]")
    return sub, slice(rank * hq, (rank + 1) * hq), slice(rank * hk, (rank + 1) * hk)


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """MAX all-reduce of a per-rank time (the job is as slow as its slowest rank)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Aggregate rate of `world` ranks that each processed `units_per_rank` in `seconds` (max over ranks)."""
    return world * units_per_rank / seconds
