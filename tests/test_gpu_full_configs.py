"""The full-size workloads (training-shape prefill, long-sequence prefill, batched decode chain, forward+backward)
run on the GPU in the launch configuration the benchmark times.  The prefill and backward shapes are compared with the
fp64 oracle on every head and sequence; the decode chain on three heads and 64 sequences spread over the batch tiles
(heads are independent -- block-diagonal gates, depthwise conv, diagonal recurrence -- and so are sequences, so the
oracle of a slice is the slice of the oracle)."""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import assert_close, f64, to_dev, to_np

pytestmark = pytest.mark.gpu


def _oracle_slice(oracle, inp, heads, batches=None):
    sl = synth.head_slice(inp, heads, batches)
    return oracle.prefill(sl["x"].astype(np.float64), f64(sl["params"]), sl["H"], c=sl["c"]), sl


def _channels(inp, heads):
    Dh = inp["D"] // inp["H"]
    return np.concatenate([np.arange(k * Dh, (k + 1) * Dh) for k in heads])


def test_config1_training_shape_prefill(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_config(1)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    y, hT, cso = binding.prefill(to_dev(inp["x"], "bf16"), params)
    torch.cuda.synchronize()
    yr, hr, cr = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), inp["H"], c=inp["c"])   # all ten heads
    assert_close("y", to_np(y), yr, "bf16")
    assert_close("h_T", to_np(hT), hr, "bf16")
    assert np.array_equal(to_np(cso), cr)
    # what holds at any size: the conv state is the last three input rows, bit for bit, for every channel
    assert np.array_equal(to_np(cso), inp["x"][:, -3:, :].astype(np.float64))
    assert torch.isfinite(y.float()).all()


def test_config2_long_sequence_prefill_with_long_memory_channels(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_config(2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    shape = binding.make_shape(1, inp["T"], inp["D"], inp["H"], torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, x.device)
    y, hT, cso = binding.prefill(x, params, workspace=ws)
    assert binding.query_status(ws) == binding.OK
    # long-memory channels (a^c = 0.9999) are spread over the heads: the carry matters over tens of thousands of tokens
    assert int((inp["params"]["lam"] > 11.0).sum()) > 100
    # all sixteen heads, four at a time (the fp64 copies of a quarter of the activations are 0.5 GB each)
    for h0 in range(0, inp["H"], 4):
        heads = list(range(h0, h0 + 4))
        ch = _channels(inp, heads)
        (yr, hr, cr), _ = _oracle_slice(oracle, inp, heads)
        chd = torch.from_numpy(ch).to(y.device)
        assert_close(f"y heads {heads}", to_np(y[:, :, chd]), yr, "bf16")
        assert_close(f"h_T heads {heads}", to_np(hT[:, chd]), hr, "bf16")
        assert np.array_equal(to_np(cso[:, :, chd]), cr)
    assert torch.isfinite(y.float()).all()


def test_config3_batched_decode_chain(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    cfg = synth.CONFIGS[3]
    T0, steps = cfg["prefill_T"], cfg["decode_steps"]
    inp = synth.make_config(3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    B, D, H = inp["B"], inp["D"], inp["H"]
    x = to_dev(inp["x"], "bf16")
    _, h, cs = binding.prefill(x[:, :T0].contiguous(), params)
    shape = binding.make_shape(B, 1, D, H, torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_DECODE, x.device)
    xt = x.transpose(0, 1).contiguous()          # [T, B, D]: one contiguous [B, D] slab per step
    ys = torch.empty(steps, B, D, dtype=torch.bfloat16, device=x.device)
    for t in range(steps):
        binding.decode_step(xt[T0 + t], params, h, cs, y=ys[t], workspace=ws)
    assert binding.query_status(ws) == binding.OK
    heads, seqs = [0, 3, 9], list(range(0, B, 8))     # 64 sampled sequences, spread over the batch tiles
    ch = _channels(inp, heads)
    (yr, hr, cr), _ = _oracle_slice(oracle, inp, heads, seqs)
    got_y = to_np(ys[:, seqs][:, :, ch]).transpose(1, 0, 2)
    assert_close("y[512:768]", got_y, yr[:, T0:], "bf16")
    assert_close("h", to_np(h[seqs][:, ch]), hr, "bf16")
    assert np.array_equal(to_np(cs[seqs][:, :, ch]), cr)
    assert np.array_equal(to_np(cs), inp["x"][:, -3:, :].astype(np.float64))


def test_config4_forward_backward(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_config(4)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); dy = to_dev(inp["dy"], "bf16")
    y, _, _ = binding.prefill(x, params)
    g = binding.backward(x, params, dy, y=y)
    torch.cuda.synchronize()
    # every head, four at a time
    for h0 in range(0, inp["H"], 4):
        heads = list(range(h0, h0 + 4))
        sl = synth.head_slice(inp, heads)
        ch = _channels(inp, heads)
        gr = oracle.backward(sl["x"].astype(np.float64), f64(sl["params"]), len(heads), sl["dy"].astype(np.float64))
        assert_close(f"dx heads {heads}", to_np(g["x"][:, :, ch]), gr["x"], "bf16")
        assert_close("dconv_w", to_np(g["conv_w"][:, ch]), gr["conv_w"], "bf16")
        for k in ("conv_b", "b_a", "b_x", "lam"):
            assert_close("d" + k, to_np(g[k][ch]), gr[k], "bf16")
        for k in ("W_a", "W_x"):
            assert_close("d" + k, to_np(g[k][h0:h0 + 4]), gr[k], "bf16")
