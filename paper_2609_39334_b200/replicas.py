"""Multi-GPU = independent replicas.  The hot path shards by problem with no exchange step (deduplication is scoped
by the context key, attention and top-k by problem), so N GPUs run N replicas of the workload on disjoint problems:
one process per GPU, no collective on the data path.  torch.distributed is used for two things only - a barrier
around the timed region and the max over ranks of the measured time."""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_workload(make_config, cfg_idx: int, rank: int, **kw):
    """Rank r's problems: same shapes, seed shifted by the rank."""
    return make_config(cfg_idx, replica=rank, **kw)


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar (device time in ms); the plain value in a single-process run."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, ms_per_step_max: float) -> float:
    """Units all ranks processed per second, given the slowest rank's step time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank / (ms_per_step_max * 1e-3)
