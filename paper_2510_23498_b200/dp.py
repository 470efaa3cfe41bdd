"""Data-parallel plumbing of the benchmark: the batch dimension shards, nothing else does.

Samples are independent through the forward loop (Alg. 1) and in the adjoint a (Alg. 2); only dL/dtheta sums over
samples.  So every rank integrates its own batch and one all-reduce (sum) of the parameter gradient per pass is the
only exchange.  With a loss that is a mean over the global batch, the caller's dL/dy_T already carries the 1/B_global
factor and the summed gradient equals the single-process one.
"""
from __future__ import annotations

import numpy as np


def shard_rows(n_rows: int, rank: int, world: int):
    """Contiguous, nearly equal row ranges: the first n_rows % world ranks get one row more."""
    base, extra = divmod(n_rows, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_sum_(tensor, world: int):
    """In-place sum over ranks of a torch tensor (NCCL on GPUs, gloo on CPU); a no-op for one rank."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(tensor, op=dist.ReduceOp.SUM)
    return tensor


def allreduce_max_float(value: float, world: int, device=None) -> float:
    """Max over ranks of a host float (used for the timed region: the slowest rank defines the step time)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
