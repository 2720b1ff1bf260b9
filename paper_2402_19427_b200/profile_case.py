"""Runs one op of the library a few times on a seeded synthetic workload; meant to be wrapped in ncu.

    python -m paper_2402_19427_b200.profile_case --op prefill --B 8 --T 2048 --D 2560 --H 10 --iters 3
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding, inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="prefill", choices=["prefill", "decode", "backward"])
    ap.add_argument("--B", type=int, default=8)
    ap.add_argument("--T", type=int, default=2048)
    ap.add_argument("--D", type=int, default=2560)
    ap.add_argument("--H", type=int, default=10)
    ap.add_argument("--io", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--generic", action="store_true")
    a = ap.parse_args()
    dt = torch.bfloat16 if a.io == "bf16" else torch.float32
    flags = binding.FLAG_FORCE_GENERIC if a.generic else 0
    p = inputs.make_inputs(1, 4, a.D, a.H, io=a.io, seed=1)["params"]
    params = binding.Params.from_numpy(p, a.io)
    g = torch.Generator(device="cuda"); g.manual_seed(0)
    if a.op == "decode":
        x = torch.randn(a.B, a.D, device="cuda", generator=g).to(dt)
        h = torch.randn(a.B, a.D, device="cuda", generator=g)
        cs = torch.randn(a.B, 3, a.D, device="cuda", generator=g).to(dt)
        for _ in range(a.iters):
            binding.decode_step(x, params, h, cs, flags=flags)
    else:
        xs = [torch.randn(a.B, a.T, a.D, device="cuda", generator=g).to(dt) for _ in range(2)]
        ys = [torch.empty_like(xs[0]) for _ in range(2)]
        if a.op == "prefill":
            shape = binding.make_shape(a.B, a.T, a.D, a.H, dt, flags=flags)
            ws = binding.alloc_workspace(shape, binding.OP_PREFILL, xs[0].device)
            for i in range(a.iters):
                binding.prefill(xs[i % 2], params, y=ys[i % 2], workspace=ws, flags=flags)
            st = binding.query_status(ws)
            assert st == binding.OK, st
        else:
            for i in range(a.iters):
                binding.backward(xs[i % 2], params, ys[0].normal_(), flags=flags)
    torch.cuda.synchronize()
    print("ok")


if __name__ == "__main__":
    main()
