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
        assert slowest == 10.0 + world - 1
        assert len(set(seeds)) == world
        print("MULTIRANK_OK")
    else:
        assert slowest == 10.0 + world - 1
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
