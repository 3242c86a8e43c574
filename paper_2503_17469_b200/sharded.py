"""Parameter-range sharding of the synchronous step for one rank per GPU.

Every element of the step is independent, so K workers on ``world`` GPUs can run Algorithm 1's
AllReduce + update as a reduce-scatter: rank r owns a contiguous range of every bucket
(``omni_shard_range``), runs the fused step on that range over all K gradient buffers -- its own
and the peer-mapped ones -- and the ranks then exchange the updated ranges and add their squared
norms.  This module holds the marshalling for that:

* range views and the sub-range ``BucketSet`` (``owned_ranges``, ``shard_buckets``);
* mapping the other ranks' buffers into this process (``map_peers``: CUDA IPC handles passed
  through ``torch.distributed``; the library's kernels then read the peers' gradients through
  those pointers with their ordinary and non-multicast bulk loads);
* the exchange of the updated ranges, in two forms: ``pull_ranges`` (device copies out of the
  peers' mapped buffers) and ``all_gather_ranges`` (one all-gather per tensor over unit-padded
  ranges through ``torch.distributed``: NCCL on GPUs, gloo with CPU tensors in the tests);
* ``total_sqnorm``: the sum of the per-rank squared norms.

The arithmetic stays in the library's kernels; nothing here computes.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

from . import binding as B

UNIT = 64  # OMNI_SHARD_UNIT: ranges are whole units, so every range starts on a 256-byte boundary of a float buffer


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


# ------------------------------------------------------------------------------------------------
# Peer mapping (CUDA IPC)
# ------------------------------------------------------------------------------------------------

def export_cuda(t):
    """A picklable description of a CUDA tensor's memory (an IPC handle plus offsets) that another
    process on the same node can open with ``open_cuda``.  The exporting process must keep the
    tensor alive for as long as any other process uses the mapping."""
    from torch.multiprocessing.reductions import reduce_tensor

    _, desc = reduce_tensor(t)
    return desc


def open_cuda(desc):
    """Map the memory described by another process's ``export_cuda`` into this process."""
    from torch.multiprocessing.reductions import rebuild_cuda_tensor

    return rebuild_cuda_tensor(*desc)


def map_peers(local: Sequence, dist, group=None) -> List[List]:
    """Every rank passes a list of its CUDA tensors (the same count and order on all ranks); the
    result is ``view[r][i]`` = rank r's i-th tensor as seen from this process: the local tensor
    for this rank, an IPC mapping for every other rank.  Collective over ``group``."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    descs = [export_cuda(t) for t in local]
    gathered = [None] * world
    dist.all_gather_object(gathered, descs, group=group)
    return [list(local) if r == rank else [open_cuda(d) for d in gathered[r]] for r in range(world)]


def pull_ranges(own: Sequence, views: Sequence[Sequence], world: int, rank: int) -> None:
    """Copy, for every tensor i and every other rank j, the range that j owns (and has just
    updated) out of j's mapped tensor ``views[j][i]`` into this rank's ``own[i]``: the all-gather
    of the updated ranges as plain device copies on the current stream.  The caller orders it
    after the owners' steps (a host barrier after their streams are synchronised)."""
    for i, t in enumerate(own):
        for j in range(world):
            if j == rank:
                continue
            b, c = B.shard_range(t.numel(), world, j)
            if c:
                t[b:b + c].copy_(views[j][i][b:b + c])


# ------------------------------------------------------------------------------------------------
# Exchange through torch.distributed
# ------------------------------------------------------------------------------------------------

def all_gather_ranges(tensors: Sequence, world: int, rank: int, dist, group=None) -> None:
    """All-gather of the updated ranges, in place, one collective per tensor: after the call every
    rank holds every range of every tensor in ``tensors`` (each a whole bucket buffer of which
    this rank has updated its own range).  The ranges differ in length by at most one unit, so
    each rank contributes its range padded to the longest one; the padding is dropped when the
    pieces are copied back."""
    import torch

    for t in tensors:
        n = t.numel()
        ranges = [B.shard_range(n, world, r) for r in range(world)]
        pad = max(c for _, c in ranges)
        if pad == 0:
            continue
        send = torch.zeros(pad, dtype=t.dtype, device=t.device)
        b, c = ranges[rank]
        send[:c].copy_(t[b:b + c])
        recv = torch.empty(world * pad, dtype=t.dtype, device=t.device)
        dist.all_gather_into_tensor(recv, send, group=group)
        for r, (rb, rc) in enumerate(ranges):
            if r != rank and rc:
                t[rb:rb + rc].copy_(recv[r * pad:r * pad + rc])


def exchange(tensors: Sequence, world: int, dist, group=None) -> None:
    """The same all-gather as one broadcast per (tensor, owner); kept for process groups without
    ``all_gather_into_tensor``.  2 x buckets x world small collectives per step: use
    ``all_gather_ranges`` where the backend has it."""
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
