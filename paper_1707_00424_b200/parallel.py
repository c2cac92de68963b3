"""Replica sharding across GPUs (one process per GPU).

Within a round the replicas never interact (Eq. parle_y .. parle_xa involve replica a and the
fixed xbar only); the single exchange of the method is the replica mean (Eq. parle_x), once per L
minibatches -- the reduce + broadcast of Section 4.1.  Every rank holds the same number of replicas,
runs its rounds with the single-GPU library and then averages the per-rank means: with equal counts
the mean of the means is the mean over all replicas."""
from __future__ import annotations

import torch
import torch.distributed as dist


def allreduce_mean_(xbar: torch.Tensor) -> torch.Tensor:
    """In place: xbar <- mean over ranks of xbar.  No-op without an initialised process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return xbar
    if dist.get_backend() == "nccl":
        dist.all_reduce(xbar, op=dist.ReduceOp.AVG)
    else:                                   # gloo has no AVG
        dist.all_reduce(xbar, op=dist.ReduceOp.SUM)
        xbar.div_(dist.get_world_size())
    return xbar
