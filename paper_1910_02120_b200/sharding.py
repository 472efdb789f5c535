"""Subnets trained on several GPUs, one process each (paper Sec. 2.1 / 2.3: each subnet goes to
a site, is trained there without communication, and only its slices travel back).

Every rank holds the full network and draws the same partition; rank r trains subnets
[r * S / world, (r + 1) * S / world) and after the local steps the ranks all-gather the trained
packed slices, so that each rank can write all S subnets back into its copy.  This is the one
exchange of a round; there is no collective inside the local steps.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch
import torch.distributed as dist


def subnet_range(S: int, world: int, rank: int) -> Tuple[int, int]:
    """(first, count) of the subnets rank `rank` trains.  S must be a multiple of world: the
    all-gather moves equal slabs."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank outside the world")
    if S % world != 0:
        raise ValueError(f"S = {S} subnets cannot be split evenly over {world} ranks")
    count = S // world
    return rank * count, count


def exchange_slices(packed: Sequence[torch.Tensor], first: int, count: int, group=None) -> int:
    """All-gathers every tensor of `packed` ([S][...] each, subnet-major) over its first dimension:
    this rank contributes slabs first .. first+count-1, afterwards every rank holds all S.
    Returns the number of bytes this rank received."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    received = 0
    for t in packed:
        if t.shape[0] != count * world:
            raise ValueError("packed tensor does not hold count * world subnets")
        if world == 1:
            continue
        flat = t.view(t.shape[0], -1)
        mine = flat[first:first + count].clone()       # the send buffer must not alias the result
        dist.all_gather_into_tensor(flat.view(-1), mine.view(-1), group=group)
        received += (world - 1) * mine.numel() * mine.element_size()
    return received


def sharded_round(ctx, seed: int, X, y, lr: float, K: int, batch: int, first: int, count: int, group=None,
                  loss_out=None, want_loss=True):
    """One IST round with this rank's share of the subnets: X, y hold the rows of the local
    subnets only ([count][K][batch] order).  ctx must have set_subnet_range(first, count) and
    work on torch's current stream (the collective is ordered after the local steps there)."""
    ctx.partition(seed)
    loss = ctx.local_steps(X, y, lr, K, batch, loss_out=loss_out, want_loss=want_loss)
    views = []
    for l in range(1, ctx.t + 1):
        views.extend(ctx.packed_layer(l))
    exchange_slices(views, first, count, group)
    ctx.reassemble()
    return loss
