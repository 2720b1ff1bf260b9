"""Partitioning of the temporal core across ranks.  No data-path collective exists: sequences are independent,
and channels are independent outside a gate block (block-diagonal W_a / W_x, depthwise conv, diagonal recurrence;
Section 4.1 of the paper, "Model parallelism"), so a rank owns whole sequences or whole heads and never exchanges activations.
The only reductions are bookkeeping (the maximum of the per-rank step time).  numpy / torch.distributed only.
"""
from __future__ import annotations

import numpy as np


def split_range(n: int, world: int, rank: int):
    """Contiguous shard [start, start + count) of n items for `rank` of `world`; sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def shard_batch(arrays: dict, world: int, rank: int) -> dict:
    """Rows [start, start+count) of every per-sequence array (x, dy, h0, conv_state); parameters are replicated."""
    B = arrays["x"].shape[0]
    s, c = split_range(B, world, rank)
    out = dict(arrays)
    for k in ("x", "dy", "h0", "conv_state"):
        if k in arrays:
            out[k] = np.ascontiguousarray(arrays[k][s:s + c])
    out["B"] = c
    return out


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's own synthetic batch in weak-scaling runs (distinct per rank, reproducible)."""
    return int(base_seed) + 1000 * int(rank)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Maximum of a scalar over all ranks (the step time of a multi-GPU run is the slowest rank's)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
