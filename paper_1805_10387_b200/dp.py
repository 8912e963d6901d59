"""Data-parallel plumbing for the step (the paper's Section 4: replicas that exchange gradients).

Rows are sharded over ranks, weights are replicated, and the only exchange is one all-reduce
(sum) of the flat FP16 weight-gradient buffer between the backward products and the update.
The update then inspects the REDUCED gradients on every rank, so all ranks take the same skip
decision and keep identical master weights without a second collective: an inf or NaN on one
rank survives the sum.  No arithmetic of the method lives here.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(M: int, rank: int, world: int):
    """Contiguous row range [lo, hi) of rank `rank`; sizes differ by at most one row."""
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_gradients(flat: torch.Tensor, group=None):
    """Sums the flat gradient buffer over the ranks in place (NCCL on GPUs, gloo on CPU)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    return flat
