"""Host-side helpers for running the sampled backward as data-parallel replicas (one process per
GPU): which synthetic batches a rank owns, and how per-rank times combine into the job's metric.
The paper's data-parallel runs sample per replica (App. C); there is no data-path exchange here."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_batches(rank: int, n_batches: int) -> list[int]:
    """Batch ids drawn by `rank`: disjoint across ranks, so replicas never share a mini-batch."""
    return [rank * n_batches + b for b in range(n_batches)]


def max_over_ranks(ms: float, device=None) -> float:
    """The slowest rank's time (the job is as slow as its slowest replica)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def ms_per_layer(ms_per_step: float, calls_per_step: int, world: int) -> float:
    """Whole-job milliseconds per layer backward: `world` replicas each finish `calls_per_step`
    backward calls in `ms_per_step` (weak scaling: the work per GPU is fixed)."""
    return ms_per_step / (calls_per_step * world)
