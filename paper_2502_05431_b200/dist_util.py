"""Host-side helpers for runs with one process per GPU.  The attention path shards by request (independent
replicas, no data-path collective); the only exchange is the timing reduction below."""
from __future__ import annotations

from typing import List, Sequence

import torch


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> List[float]:
    """Element-wise maximum of a list of per-rank numbers over all ranks (identity without a process group)."""
    import torch.distributed as td
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if td.is_available() and td.is_initialized() and td.get_world_size() > 1:
        td.all_reduce(t, op=td.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank: float, world_size: int, slowest_rank_ms: float) -> float:
    """Aggregate throughput of `world_size` replicas that each processed `units_per_rank` units: all units over the
    time of the slowest rank (units per second)."""
    return world_size * units_per_rank / (slowest_rank_ms * 1e-3)


def replica_seed(base_seed: int, rank: int) -> int:
    """Every rank works on its own, differently seeded replica of the workload."""
    return base_seed + 100 * rank
