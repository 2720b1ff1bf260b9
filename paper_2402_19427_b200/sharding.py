"""Partitioning of the temporal core across ranks.  Sequences are independent, and channels are independent outside a
gate block (block-diagonal W_a / W_x, depthwise conv, diagonal recurrence; Section 4.1 of the paper, "Model parallelism"),
so a rank that owns whole sequences or whole heads never exchanges activations; the only reduction there is bookkeeping
(the maximum of the per-rank step time).

A sequence may also be split along time, rank r owning tokens [t_r, t_r + T_r).  Eq. 4 is affine in the incoming state, so a
rank's share of the sequence acts on the state as one step h_out = A_r h_in + b_r with A_r = prod_t a_t and b_r its final
state from a zero start; these steps compose as (A_2 A_1, A_2 b_1 + b_2).  Two small messages per rank suffice: the last
three raw inputs of the share (the Conv1D history of the next rank), and the pair (A_r, b_r).  Every rank then knows its
incoming state and runs the real forward (prefill_time_share).  numpy / torch.distributed only, apart from that function's
calls into the CUDA binding; no arithmetic of Eq. 1-3 lives here.
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


def combine_steps(first, second):
    """Composition of two affine steps h -> A h + b applied in this order: (A_2 A_1, A_2 b_1 + b_2).  Works on numpy arrays
    and torch tensors alike; associative, with identity (1, 0)."""
    a1, b1 = first
    a2, b2 = second
    return a2 * a1, a2 * b1 + b2


def exchange_conv_history(x_tail, dist, conv_state_in=None):
    """The Conv1D history of this rank's time share: the last three raw inputs [B,3,D] of the rank before it
    (`conv_state_in`, or zeros, for rank 0).  `x_tail` is this rank's own last three rows; every share must hold at
    least three tokens.  One all-gather of [B,3,D] per rank."""
    import torch
    if x_tail.shape[1] != 3:
        raise ValueError("x_tail must be the last three token rows of this rank's share")
    rank, world = dist.get_rank(), dist.get_world_size()
    tails = [torch.empty_like(x_tail) for _ in range(world)]
    dist.all_gather(tails, x_tail.contiguous())
    if rank > 0:
        return tails[rank - 1]
    return conv_state_in if conv_state_in is not None else torch.zeros_like(x_tail)


def exchange_time_steps(a_prod, h_end, dist, h0=None):
    """Incoming recurrent state [B,D] of this rank's time share.  `a_prod`, `h_end` [B,D]: the rank's share as one affine
    step (prod_t a_t, and the final state of a forward from a zero state with the right Conv1D history).  One all-gather of
    [B,2,D] per rank, then the exclusive scan over ranks of `combine_steps`, applied to `h0` (zeros if None)."""
    import torch
    rank, world = dist.get_rank(), dist.get_world_size()
    mine = torch.stack([a_prod, h_end], dim=1).contiguous()
    steps = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(steps, mine)
    h = h0.clone() if h0 is not None else torch.zeros_like(h_end)
    for r in range(rank):
        h = steps[r][:, 0] * h + steps[r][:, 1]
    return h


def prefill_time_share(x_share, params, dist, h0=None, conv_state_in=None, c=8.0, workspace=None):
    """This rank's share of a prefill whose sequences are split along time: rank r holds tokens [t_r, t_r + T_r) of every
    sequence as `x_share` [B,T_r,D] on its GPU (T_r >= 3), `params` is the layer on that GPU, `h0` / `conv_state_in` are
    the state before the first token of the whole sequence (used by rank 0's share).  Two small all-gathers and two runs
    of the kernel: the first from a zero state, which yields the share as one affine step (prod_t a_t, h_end), the second
    from the incoming state that the exclusive scan over the ranks' steps gives.  Rank 0 starting from a zero state needs
    only the first run.  Returns (y [B,T_r,D], h_end [B,D], conv_state [B,3,D]); the last rank's h_end and conv_state are
    those of the whole sequence.  Imports the CUDA binding: there is no CPU path."""
    import torch
    from . import binding
    B, T_r, D = x_share.shape
    if T_r < 3:
        raise ValueError("every time share must hold at least three tokens")
    hist = exchange_conv_history(x_share[:, -3:].contiguous(), dist, conv_state_in)
    a_prod = torch.empty(B, D, dtype=torch.float32, device=x_share.device)
    y, h_zero, cs = binding.prefill(x_share, params, conv_state_in=hist, c=c, workspace=workspace, a_prod=a_prod)
    h_in = exchange_time_steps(a_prod, h_zero, dist, h0)
    if dist.get_rank() == 0 and h0 is None:
        return y, h_zero, cs
    return binding.prefill(x_share, params, h0=h_in, conv_state_in=hist, c=c, workspace=workspace, y=y)
