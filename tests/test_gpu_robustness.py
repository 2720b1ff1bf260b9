"""What the parity tests do not show: nothing is written outside the output buffers (guard bytes around every output and
around the workspace), a bounded device-side wait that runs out ends in RGLRU_ERR_TIMEOUT with the context still usable,
and a head shard run on its own reproduces the same channels of the full run bit for bit (Section 4.1: the block-diagonal
gates make heads independent, so tensor-parallel ranks own heads without exchanging anything)."""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import Guarded, assert_close, f64, oracle_prefill, to_dev, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,T,H", [(1, 1, 1), (2, 65, 1), (3, 129, 2), (1, 1000, 1), (8, 320, 3)])
def test_prefill_writes_only_its_outputs(oracle, B, T, H):
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=900 + T, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    shape = binding.make_shape(B, T, D, H, torch.bfloat16)
    g = Guarded()
    y = g.empty((B, T, D), torch.bfloat16)
    hT = g.empty((B, D), torch.float32)
    cso = g.empty((B, 3, D), torch.bfloat16)
    ws = g.empty((binding.workspace_bytes(shape, binding.OP_PREFILL),), torch.uint8)
    ws.zero_()
    binding.prefill(x, params, h0=to_dev(inp["h0"]), conv_state_in=to_dev(inp["conv_state"], "bf16"), y=y, h_T=hT,
                    conv_state_out=cso, workspace=ws)
    g.check()
    assert binding.query_status(ws) == binding.OK
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", to_np(y), yr, "bf16"); assert_close("h_T", to_np(hT), hr, "bf16")
    assert np.array_equal(to_np(cso), cr)


@pytest.mark.parametrize("B,H,flags", [(80, 1, 0), (37, 2, 0), (5, 1, 1)])
def test_decode_step_writes_only_its_outputs(B, H, flags):
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    inp = synth.make_inputs(B, 4, D, H, io="bf16", seed=77, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    g = Guarded()
    y = g.empty((B, D), torch.bfloat16)
    h = g.empty((B, D), torch.float32); h.copy_(to_dev(inp["h0"]))
    cs = g.empty((B, 3, D), torch.bfloat16); cs.copy_(to_dev(inp["conv_state"], "bf16"))
    shape = binding.make_shape(B, 1, D, H, torch.bfloat16, flags=flags)
    ws = g.empty((binding.workspace_bytes(shape, binding.OP_DECODE),), torch.uint8); ws.zero_()
    for t in range(3):
        binding.decode_step(to_dev(inp["x"][:, t], "bf16"), params, h, cs, y=y, workspace=ws, flags=flags)
    g.check()
    assert torch.isfinite(y.float()).all() and torch.isfinite(h).all()


@pytest.mark.parametrize("B,T,H,io,flags", [(2, 64, 1, "bf16", 0), (1, 200, 2, "bf16", 0), (2, 70, 2, "f32", 1)])
def test_backward_writes_only_its_outputs(B, T, H, io, flags):
    import torch
    from paper_2402_19427_b200 import binding
    D = (256 if io == "bf16" else 32) * H
    dt = torch.bfloat16 if io == "bf16" else torch.float32
    inp = synth.make_inputs(B, T, D, H, io=io, seed=55, with_dy=True)
    params = binding.Params.from_numpy(inp["params"], io)
    x = to_dev(inp["x"], io); dy = to_dev(inp["dy"], io)
    Dh = D // H
    g = Guarded()
    f32 = torch.float32
    out = dict(x=g.empty((B, T, D), dt), conv_w=g.empty((4, D), f32), conv_b=g.empty((D,), f32), W_a=g.empty((H, Dh, Dh), f32),
               b_a=g.empty((D,), f32), W_x=g.empty((H, Dh, Dh), f32), b_x=g.empty((D,), f32), lam=g.empty((D,), f32))
    shape = binding.make_shape(B, T, D, H, dt, flags=flags)
    ws = g.empty((binding.workspace_bytes(shape, binding.OP_BACKWARD),), torch.uint8); ws.zero_()
    binding.backward(x, params, dy, flags=flags, workspace=ws, out=out)
    g.check()
    for k, v in out.items():
        assert torch.isfinite(v.float()).all(), k


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_clean(oracle):
    """One sequence split in time over several CTA pairs: every tile after the first waits for carry records.  Under the
    test flag the records it looks for never appear, the wait limit is one millisecond, so the kernel gives up, drains and
    returns; the status word says so, and the same workspace then serves an ordinary call that matches the oracle."""
    import torch
    from paper_2402_19427_b200 import binding
    B, T, H = 1, 1024, 1
    inp = synth.make_inputs(B, T, 256 * H, H, io="bf16", seed=13)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    shape = binding.make_shape(B, T, 256 * H, H, torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, x.device)
    prev = binding.set_wait_limit_ns(1_000_000)
    try:
        binding.prefill(x, params, workspace=ws, flags=binding.FLAG_TEST_CARRY_NEVER_ARRIVES)
        torch.cuda.synchronize()
        assert binding.query_status(ws) == binding.ERR_TIMEOUT
        assert binding.query_status(ws) == binding.OK          # reported once
    finally:
        binding.set_wait_limit_ns(prev)
    y, hT, cso = binding.prefill(x, params, workspace=ws)
    torch.cuda.synchronize()
    assert binding.query_status(ws) == binding.OK
    yr, hr, cr = oracle_prefill(oracle, inp)
    assert_close("y", to_np(y), yr, "bf16"); assert_close("h_T", to_np(hT), hr, "bf16")
    assert np.array_equal(to_np(cso), cr)


def test_head_shard_reproduces_the_full_run_bit_for_bit():
    """Heads [1, 3) of a four-head layer run as their own two-head problem on the sliced tensors (what a tensor-parallel
    rank owning those heads would do).  Sequences are dealt whole to the CTA pairs in both runs, so the arithmetic per
    channel is the same and the results must be identical bits."""
    import torch
    from paper_2402_19427_b200 import binding
    B, T, H = 16, 200, 4
    inp = synth.make_inputs(B, T, 256 * H, H, io="bf16", seed=21, with_state=True, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    y, hT, cso = binding.prefill(to_dev(inp["x"], "bf16"), params, h0=to_dev(inp["h0"]),
                                 conv_state_in=to_dev(inp["conv_state"], "bf16"))
    heads = [1, 2]
    sl = synth.head_slice(inp, heads)
    ch = np.arange(256 * heads[0], 256 * (heads[-1] + 1))
    ps = binding.Params.from_numpy(sl["params"], "bf16")
    ys, hs, cs = binding.prefill(to_dev(sl["x"], "bf16"), ps, h0=to_dev(inp["h0"][:, ch]),
                                 conv_state_in=to_dev(inp["conv_state"][:, :, ch], "bf16"))
    torch.cuda.synchronize()
    chd = torch.from_numpy(ch).to(y.device)
    assert torch.equal(ys, y[:, :, chd]) and torch.equal(hs, hT[:, chd]) and torch.equal(cs, cso[:, :, chd])
