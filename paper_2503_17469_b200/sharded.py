"""Parameter-range sharding of the synchronous step for one rank per GPU.

Every element of the step is independent, so K workers on ``world`` GPUs can run Algorithm 1's
AllReduce + update as a reduce-scatter: rank r owns a contiguous range of every bucket
(``omni_shard_range``), runs the fused step on that range over all K gradient buffers -- its own
and the peer-mapped ones -- and the ranks then exchange the updated ranges and add their squared
norms.  This module holds the marshalling for that: range views, the sub-range ``BucketSet`` and
the exchange through ``torch.distributed`` (NCCL on GPUs; the same calls run on gloo with CPU
tensors, which is how the protocol is tested without several GPUs).  The arithmetic stays in the
library's kernels; nothing here computes.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

from . import binding as B


def owned_ranges(numels: Sequence[int], world: int, rank: int):
    """[(begin, count)] per bucket for this rank."""
    return [B.shard_range(int(n), world, rank) for n in numels]


def shard_buckets(params: Sequence, grads: Sequence[Sequence], momenta: Optional[Sequence], params_lp: Optional[Sequence],
                  world: int, rank: int) -> B.BucketSet:
    """The ``BucketSet`` of the ranges rank ``rank`` owns: views into the given per-bucket tensors
    (``grads[i][k]`` = worker k's gradient of bucket i, local or peer-mapped).  Buckets of which
    the rank owns nothing stay in the set with zero elements (the library skips them)."""
    rng = owned_ranges([p.numel() for p in params], world, rank)
    cut = lambda t, i: t[rng[i][0]:rng[i][0] + rng[i][1]]
    return B.BucketSet([cut(p, i) for i, p in enumerate(params)],
                       [[cut(g, i) for g in row] for i, row in enumerate(grads)],
                       [cut(m, i) for i, m in enumerate(momenta)] if momenta is not None else None,
                       [cut(lp, i) for i, lp in enumerate(params_lp)] if params_lp is not None else None)


def exchange(tensors: Sequence, world: int, dist, group=None) -> None:
    """All-gather of the updated ranges, in place: after the call every rank holds every range
    of every tensor in ``tensors`` (each a whole bucket buffer of which this rank has updated its
    own range).  One broadcast per (bucket, owner): the ranges differ in length by up to one
    unit, so they are sent as they are instead of being padded to a common size."""
    for t in tensors:
        for owner in range(world):
            b, c = B.shard_range(t.numel(), world, owner)
            if c:
                dist.broadcast(t[b:b + c], src=owner, group=group)


def total_sqnorm(local_sqnorm: float, dist, device=None, group=None) -> float:
    """Sum over ranks of the squared norms of their ranges = the squared norm of the aggregate."""
    import torch

    x = torch.tensor([local_sqnorm], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(x, op=dist.ReduceOp.SUM, group=group)
    return float(x.item())
