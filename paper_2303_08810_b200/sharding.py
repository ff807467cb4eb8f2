"""Batch sharding of BRA over ranks (one process per GPU).

Every image is independent in the forward pass, and so are dQ, dK, dV in the
backward pass: ranks split the batch and exchange nothing.  Only the LCE
weight / bias gradients sum over the batch, so they need one small all-reduce
after the local `bra_backward` calls.  No arithmetic of the method lives here.
"""
from __future__ import annotations


def shard_range(B: int, world: int, rank: int) -> tuple[int, int]:
    """Images [lo, hi) of a batch of B owned by `rank`: contiguous, sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_lce_grads(d_lce_w, d_lce_b=None, group=None):
    """Sum the LCE weight (and bias) gradients of all ranks in place; returns them.

    Works on whatever device the tensors live on (NCCL for CUDA tensors, gloo for CPU).
    A rank whose shard is empty passes zeros.
    """
    import torch.distributed as dist
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return d_lce_w, d_lce_b
    dist.all_reduce(d_lce_w, op=dist.ReduceOp.SUM, group=group)
    if d_lce_b is not None:
        dist.all_reduce(d_lce_b, op=dist.ReduceOp.SUM, group=group)
    return d_lce_w, d_lce_b


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Largest `value` over the ranks (timings of a step are reported as the slowest rank's)."""
    import torch
    import torch.distributed as dist
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
