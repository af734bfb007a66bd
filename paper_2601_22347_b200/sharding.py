"""Row sharding of the PeRQ online path across ranks (one process per GPU).

Token rows are independent (the rotation and the permutation act on the channel dimension
only), so `perq_rotate_quantize` shards over T with no data-path collective: every rank
runs the call on its own contiguous rows and the outputs are disjoint row ranges.  Only
the calibration statistic needs an exchange when its rows are sharded: the per-channel
sums add up, the per-block means are averaged with the ranks' row counts as weights, and
the per-token maxima stay local.  This module holds that host-side logic; it works on CPU
tensors with the `gloo` backend and on CUDA tensors with `nccl`.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch


def row_shard(T: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced row range [start, stop) of `rank`; the first T % world ranks get one row more."""
    assert 0 <= rank < world and T >= 0
    base, extra = divmod(T, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a multi-rank step costs."""
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def allreduce_block_l1_stats(chan_abs_sum: Optional[torch.Tensor], block_l1_mean: Optional[torch.Tensor],
                             rows_local: int):
    """Combine the statistic of row shards in place: channel sums are added, block means are
    averaged weighted by the ranks' row counts.  Returns the total number of rows."""
    import torch.distributed as dist
    ref = chan_abs_sum if chan_abs_sum is not None else block_l1_mean
    device = ref.device if ref is not None else "cpu"
    n = torch.tensor([float(rows_local)], dtype=torch.float64, device=device)
    if not (dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1):
        return int(rows_local)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    total = float(n.item())
    if chan_abs_sum is not None:
        dist.all_reduce(chan_abs_sum, op=dist.ReduceOp.SUM)
    if block_l1_mean is not None:
        block_l1_mean.mul_(float(rows_local))
        dist.all_reduce(block_l1_mean, op=dist.ReduceOp.SUM)
        block_l1_mean.div_(total)
    return int(total)
