"""Data-parallel use of the layer: shard the batch, keep the probes identical, sum the estimates.

The sketch is independent per sample (column b of S needs only X[b]), the back-probe sums over the
local samples and the contraction is linear in L, so each rank produces a partial dW estimate from
its own samples with the SAME Z, and one all-reduce(sum) of dW (Cout*Cin*KH*KW floats) completes the
layer -- the same exchange ordinary data-parallel training already does for gradients.  Y and dX are
per sample and need no communication.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def batch_shard(global_batch: int, rank: int, world: int) -> tuple[int, int]:
    """[start, stop) of the samples rank ``rank`` owns; shards differ by at most one sample."""
    base, extra = divmod(global_batch, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_dw(dW: torch.Tensor, group=None) -> torch.Tensor:
    """Sum the per-rank dW estimates in place (no-op without an initialised process group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
    return dW
