"""Row sharding of the weight path over several GPUs (one process per GPU).

Every quantity of the path depends on one output channel only: alpha, z, the codes, the slices, the packed rows, the
overflow lists and y[:, n] are functions of row n of W.  Partitioning by output channel therefore needs no exchange
inside the path; x is replicated and, if every rank wants the whole y, one all-gather of B * N / G floats per rank
finishes the layer.  These helpers hold that host-side logic; they work with any torch.distributed backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_range(N: int, world: int, rank: int, multiple: int = 16):
    """Rows [lo, hi) of an N-row matrix owned by `rank`: contiguous blocks whose sizes are multiples of `multiple`
    (the kernels' row-tile granularity) except possibly the last non-empty one."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad world / rank")
    blocks = (N + multiple - 1) // multiple
    per, extra = divmod(blocks, world)
    lo_b = rank * per + min(rank, extra)
    hi_b = lo_b + per + (1 if rank < extra else 0)
    return min(lo_b * multiple, N), min(hi_b * multiple, N)


def all_gather_rows(y_local: torch.Tensor, N: int, group=None, multiple: int = 16) -> torch.Tensor:
    """y_local: [B, rows of this rank] -> [B, N] on every rank.  Shards may differ in width, so every rank sends a
    buffer padded to the widest shard."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    ranges = [row_range(N, world, r, multiple) for r in range(world)]
    lo, hi = ranges[rank]
    if y_local.shape[1] != hi - lo:
        raise ValueError("y_local does not match this rank's row range")
    widest = max(h - l for l, h in ranges)
    send = y_local.new_zeros((y_local.shape[0], widest))
    send[:, : hi - lo] = y_local
    recv = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(recv, send, group=group)
    out = y_local.new_empty((y_local.shape[0], N))
    for (l, h), part in zip(ranges, recv):
        out[:, l:h] = part[:, : h - l]
    return out
