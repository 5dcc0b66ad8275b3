"""Host-side helpers for running the sampled backward as data-parallel replicas (one process per
GPU): which synthetic batches a rank owns, how per-rank times combine into the job's metric, and the
sum of the replicas' parameter gradients.  The paper's data-parallel runs sample per replica (App. C):
the sampled backward itself needs no exchange; the only exchange of a data-parallel step is the
all-reduce of every layer's dW, which App. C names as what limits the time gained."""
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


class GradReducer:
    """Sums the replicas' parameter gradients, overlapped with the backward of the layers below: a layer's
    all-reduce is issued as soon as its backward call is enqueued (the collective runs on the communication
    library's own stream, ordered after the work enqueued so far), and is only waited for at the end of the
    pass, before an optimiser would read the gradients.  Every replica's estimator is unbiased for its shard,
    so the sum over replicas is unbiased for the batch (divide by the world size for the mean)."""

    def __init__(self):
        self.works = []
        self.active = dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1

    def reduce_async(self, dW: torch.Tensor) -> None:
        if self.active:
            self.works.append(dist.all_reduce(dW, op=dist.ReduceOp.SUM, async_op=True))

    def wait(self) -> None:
        for w in self.works:
            w.wait()
        self.works.clear()
