"""Host-side helpers for running N independent replicas of the path (one process per GPU).

The path shards with no exchange (independent per layer, sequence and KV head), so multi-GPU runs are
replicas: torch.distributed is used only for a barrier and to take the maximum of the device times over
ranks.  No data-path collective exists."""
from __future__ import annotations

from typing import Dict

import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(times: Dict[str, float]) -> Dict[str, float]:
    """Element-wise maximum of a dict of per-stage times over all ranks (identity for one process)."""
    if world() == 1:
        return dict(times)
    gathered = [None] * world()
    dist.all_gather_object(gathered, times)
    return {k: max(g[k] for g in gathered) for k in times}


def aggregate_throughput(units_per_rank: float, seconds_max_over_ranks: float) -> float:
    """Whole-job throughput of `world()` replicas that each processed `units_per_rank` in the given time."""
    return world() * units_per_rank / seconds_max_over_ranks
