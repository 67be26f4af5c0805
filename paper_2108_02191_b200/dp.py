"""Data-parallel training step on top of the C-ABI calls (Section 1 of the paper: the compressed
model fits every GPU, so it is trained data-parallel and the ranks exchange one gradient the
size of the array).

Every rank holds a replica of the array and a shard of the batch (split by sample).  One step:

    robe_backward   this rank's scatter-add into a dense fp32 gradient        (this library)
    all-reduce      sum of the gradients over the ranks, 4 M bytes per rank   (torch.distributed)
    robe_apply_sgd  array <- fma(-lr, gradient, array); gradient zeroed       (this library)

All replicas apply the same sum, so they stay bit-identical.  Nothing here computes anything of
the method: the functions order library calls and one collective, and cut host-side id lists.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np


def shard_by_sample(indices: np.ndarray, offsets: Optional[np.ndarray], batch: int, num_tables: int,
                    rank: int, world: int) -> Tuple[np.ndarray, Optional[np.ndarray], int, int]:
    """Rank `rank`'s shard of a sample-major batch: samples [n0, n1), n0 = rank*batch // world.
    Returns (indices, offsets or None, n0, n1); the offsets are rebased to start at 0."""
    n0, n1 = rank * batch // world, (rank + 1) * batch // world
    b0, b1 = n0 * num_tables, n1 * num_tables
    if offsets is None:
        return np.ascontiguousarray(indices[b0:b1]), None, n0, n1
    lo, hi = int(offsets[b0]), int(offsets[b1])
    return (np.ascontiguousarray(indices[lo:hi]),
            np.ascontiguousarray(offsets[b0:b1 + 1] - lo), n0, n1)


def robe_dp_step(h, grad_out, indices, offsets, batch: int, grad_array, lr: float, workspace=None,
                 group=None, stream=None) -> None:
    """One data-parallel SGD step of this rank: backward into grad_array (which must hold zeros,
    as robe_apply_sgd leaves it), all-reduce over `group` (skipped when no process group has
    been initialised), dense apply.  The backward runs in the handle's backward mode."""
    import torch.distributed as dist

    from . import binding as robe

    robe.robe_backward(h, grad_out, indices, offsets, batch, grad_array, 0.0, workspace, stream)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(grad_array, op=dist.ReduceOp.SUM, group=group)
    robe.robe_apply_sgd(h, grad_array, lr, True, stream)


def replicas_identical(array, group=None) -> bool:
    """True when every rank's array has the same bits (compared through two integer
    all-reduces of a checksum of the bit patterns)."""
    import torch
    import torch.distributed as dist

    bits = array.view(torch.int32).to(torch.int64)
    # two sums with different weights: a swap or a single changed bit shows in at least one
    w = torch.arange(1, bits.numel() + 1, device=bits.device, dtype=torch.int64) % 65521
    check = torch.stack([bits.sum(), (bits * w).sum()])
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return True
    lo, hi = check.clone(), check.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
    return bool((lo == hi).all().item())
