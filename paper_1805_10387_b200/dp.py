"""Data-parallel plumbing for the step (the paper's Section 4: replicas that exchange gradients).

Rows are sharded over ranks and the FP16 working weights are replicated.  Two schedules for
what follows the backward products, both with one exchange of the flat FP16 gradient buffer:

replicated update   all-reduce (sum) of the gradients; every rank then runs the same fused
                    update over all parameters, inspecting the REDUCED gradients, so all ranks
                    take the same skip decision and keep identical FP32 masters without a
                    second collective (an inf or NaN on one rank survives the sum).
sharded update      reduce-scatter of the gradients: rank r receives the summed slice
                    [r n, (r + 1) n) of the flat range (n = padded total / ranks, a multiple
                    of 8 elements so that every slice starts on a 16-byte boundary); it keeps
                    the FP32 master and the moments of that slice only, inspects and updates
                    it, and an all-gather of the rewritten FP16 slices restores the full
                    working copy everywhere.  A rank sees only its slice of the sum, so the
                    ranks agree on the overflow flag with a max-reduction of one word.

This module moves data only: no arithmetic of the method lives here, and no kernel of the
library is ever handed another GPU's memory (collectives land in local buffers first).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(M: int, rank: int, world: int):
    """Contiguous row range [lo, hi) of rank `rank`; sizes differ by at most one row."""
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_params(total: int, rank: int, world: int):
    """Slice [lo, hi) of a flat parameter range of `total` elements that rank `rank` owns in the
    sharded update.  `total` must be a multiple of 8 * world, which makes the slices equal and
    16-byte aligned for FP16 and FP32 alike."""
    if total % (8 * world):
        raise ValueError(f"flat range of {total} elements is not a multiple of 8 * {world}")
    n = total // world
    return rank * n, (rank + 1) * n


def padded_total(total: int, world: int) -> int:
    """Smallest multiple of 8 * world that holds `total` elements."""
    q = 8 * world
    return (total + q - 1) // q * q


def allreduce_gradients(flat: torch.Tensor, group=None):
    """Sums the flat gradient buffer over the ranks in place (NCCL on GPUs, gloo on CPU)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    return flat


class Comm:
    """The exchanges of a data-parallel step over a torch.distributed process group."""

    def __init__(self, group=None):
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self._native_rs = dist.get_backend(group) == "nccl"      # gloo has no reduce-scatter

    def all_reduce(self, flat: torch.Tensor):
        dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=self.group)

    def reduce_scatter(self, flat: torch.Tensor, out: torch.Tensor):
        """out = sum over ranks of their flat[lo:hi], [lo, hi) = this rank's slice."""
        lo, hi = shard_params(flat.numel(), self.rank, self.world)
        assert out.numel() == hi - lo
        if self._native_rs:
            dist.reduce_scatter_tensor(out, flat, op=dist.ReduceOp.SUM, group=self.group)
        else:       # same result through an all-reduce of a copy
            tmp = flat.clone()
            dist.all_reduce(tmp, op=dist.ReduceOp.SUM, group=self.group)
            out.copy_(tmp[lo:hi])

    def all_gather(self, flat: torch.Tensor, mine: torch.Tensor):
        """flat[r n:(r + 1) n] = rank r's `mine` for every r (`mine` may be this rank's slice of flat)."""
        n = flat.numel() // self.world
        assert mine.numel() == n and flat.numel() == n * self.world
        if self._native_rs:
            dist.all_gather_into_tensor(flat, mine, group=self.group)
        else:
            parts = [torch.empty_like(mine) for _ in range(self.world)]
            dist.all_gather(parts, mine.clone(), group=self.group)
            for r, p in enumerate(parts):
                flat[r * n:(r + 1) * n].copy_(p)

    def all_reduce_max(self, word: torch.Tensor):
        dist.all_reduce(word, op=dist.ReduceOp.MAX, group=self.group)
