"""Worker of test_multirank_cpu.py: one process per rank, gloo backend, CPU only."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
from paper_2402_19427_b200 import inputs as synth, sharding  # noqa: E402


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    f64 = lambda p: {k: np.asarray(v, np.float64) for k, v in p.items()}
    # one global batch, sharded by sequence: each rank runs its rows with replicated weights, nothing is exchanged
    inp = synth.make_inputs(5, 40, 64, 2, io="bf16", seed=77, with_state=True)
    mine = sharding.shard_batch(inp, world, rank)
    y, hT, cs = oracle.prefill(mine["x"].astype(np.float64), f64(inp["params"]), 2, h0=mine["h0"].astype(np.float64),
                               conv_state_in=mine["conv_state"].astype(np.float64))
    parts = [None] * world
    dist.all_gather_object(parts, (y, hT, cs))           # test bookkeeping only: not part of the data path
    # head sharding: each rank owns whole heads (its slice of W, b, Lambda, conv taps and of the channel dimension)
    hs, hc = sharding.split_range(inp["H"], world, rank)
    sl = synth.head_slice(inp, range(hs, hs + hc))
    yh, _, _ = oracle.prefill(sl["x"].astype(np.float64), f64(sl["params"]), hc, h0=sl["h0"].astype(np.float64),
                              conv_state_in=sl["conv_state"].astype(np.float64))
    hparts = [None] * world
    dist.all_gather_object(hparts, yh)
    # time sharding: the sequence is cut along time; one message carries the Conv1D history, one the share as an affine step
    g = synth.make_inputs(3, 45, 64, 2, io="bf16", seed=78, with_state=True)
    gp = f64(g["params"])
    ts, tc = sharding.split_range(45, world, rank)
    xs = g["x"][:, ts:ts + tc].astype(np.float64)
    hist = sharding.exchange_conv_history(torch.from_numpy(np.ascontiguousarray(xs[:, -3:])), dist,
                                          conv_state_in=torch.from_numpy(g["conv_state"].astype(np.float64))).numpy()
    _, b_r, _, a_r = oracle.prefill(xs, gp, 2, conv_state_in=hist, with_a_prod=True)
    h_in = sharding.exchange_time_steps(torch.from_numpy(a_r), torch.from_numpy(b_r), dist,
                                        h0=torch.from_numpy(g["h0"].astype(np.float64))).numpy()
    yt, hTt, cst = oracle.prefill(xs, gp, 2, h0=h_in, conv_state_in=hist)
    tparts = [None] * world
    dist.all_gather_object(tparts, (yt, hTt, cst))
    slowest = sharding.max_over_ranks(10.0 + rank, dist)
    seeds = [None] * world
    dist.all_gather_object(seeds, sharding.rank_seed(synth.BASE_SEED, rank))
    if rank == 0:
        yf, hf, cf = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), 2, h0=inp["h0"].astype(np.float64),
                                    conv_state_in=inp["conv_state"].astype(np.float64))
        assert np.array_equal(np.concatenate([p[0] for p in parts], 0), yf)
        assert np.array_equal(np.concatenate([p[1] for p in parts], 0), hf)
        assert np.array_equal(np.concatenate([p[2] for p in parts], 0), cf)
        assert np.array_equal(np.concatenate(hparts, 2), yf)
        yg, hg, cg = oracle.prefill(g["x"].astype(np.float64), gp, 2, h0=g["h0"].astype(np.float64),
                                    conv_state_in=g["conv_state"].astype(np.float64))
        np.testing.assert_allclose(np.concatenate([p[0] for p in tparts], 1), yg, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(tparts[-1][1], hg, rtol=1e-12, atol=1e-14)      # the last rank ends in the final state
        assert np.array_equal(tparts[-1][2], cg)
        assert slowest == 10.0 + world - 1
        assert len(set(seeds)) == world
        print("MULTIRANK_OK")
    else:
        assert slowest == 10.0 + world - 1
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
