"""Batch sharding across GPUs: instances are independent, so rank r simply takes a contiguous
slice of the batch and no collective touches the data path.  ``gather_selection`` is an optional
convenience that concatenates per-rank results (an all-gather of B*(4n+20) bytes)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(total: int, world: int, rank: int) -> tuple[int, int]:
    """(first instance, number of instances) of ``rank``: contiguous, sizes differ by at most one."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def gather_selection(idx: torch.Tensor, barrier: torch.Tensor, wait: torch.Tensor, status: torch.Tensor,
                     total: int, group=None):
    """All ranks get the full [total, n] idx and [total] barrier / wait / status, in instance order."""
    world = dist.get_world_size(group)
    n = idx.shape[1]
    counts = [shard_range(total, world, r)[1] for r in range(world)]
    cap = max(counts)

    def pad(t, shape, dtype):
        out = torch.zeros(shape, dtype=dtype, device=t.device)
        out[: t.shape[0]] = t
        return out

    outs = []
    for t, shape in ((idx, (cap, n)), (barrier, (cap,)), (wait, (cap,)), (status, (cap,))):
        parts = [torch.empty(shape, dtype=t.dtype, device=t.device) for _ in range(world)]
        dist.all_gather(parts, pad(t, shape, t.dtype), group=group)
        outs.append(torch.cat([p[:c] for p, c in zip(parts, counts)], dim=0))
    return tuple(outs)
