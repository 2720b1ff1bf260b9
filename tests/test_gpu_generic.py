"""GPU parity of the shape-generic CUDA kernels (prefill, decode step, backward) against the fp64 oracle,
element by element on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import assert_close, f64, gpu_prefill, oracle_prefill, to_dev, to_np

pytestmark = pytest.mark.gpu
GENERIC = 1  # RGLRU_FLAG_FORCE_GENERIC


def test_config0_fp32_tiny(oracle):
    inp = synth.make_config(0)
    y, hT, cso = gpu_prefill(inp)
    yr, hr, cr = oracle_prefill(oracle, inp)
    assert_close("y", y, yr, "f32"); assert_close("h_T", hT, hr, "f32")
    assert np.array_equal(cso, cr)


@pytest.mark.parametrize("B,T,D,H,io", [
    (2, 1, 16, 2, "f32"), (1, 2, 24, 3, "f32"), (3, 3, 8, 1, "f32"), (2, 37, 96, 3, "f32"),
    (1, 100, 600, 2, "f32"),      # head width 300 > 256 threads, ragged tile tails
    (2, 50, 64, 4, "bf16"), (1, 130, 512, 2, "bf16"), (2, 17, 40, 5, "bf16"),
])
def test_prefill_shapes_with_state_and_bias(oracle, B, T, D, H, io):
    inp = synth.make_inputs(B, T, D, H, io=io, seed=100 + T, with_state=True, bias_scale=0.5)
    y, hT, cso = gpu_prefill(inp, flags=GENERIC, h0=inp["h0"], cs=inp["conv_state"])
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", y, yr, io); assert_close("h_T", hT, hr, io)
    assert np.array_equal(cso, cr)                       # raw copies: bit-exact


def test_prefill_aliased_state_and_split(oracle):
    """h_T may alias h0 and conv_state_out may alias conv_state_in; prefill(T1) then prefill(T2) == prefill(T1+T2)."""
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(2, 41, 64, 2, io="f32", seed=7, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "f32")
    x = to_dev(inp["x"])
    h = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"])
    y1, _, _ = binding.prefill(x[:, :2].contiguous(), params, h0=h, conv_state_in=cs, h_T=h, conv_state_out=cs, flags=GENERIC)
    y2, _, _ = binding.prefill(x[:, 2:].contiguous(), params, h0=h, conv_state_in=cs, h_T=h, conv_state_out=cs, flags=GENERIC)
    torch.cuda.synchronize()
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", np.concatenate([to_np(y1), to_np(y2)], 1), yr, "f32")
    assert_close("h_T", to_np(h), hr, "f32")
    assert np.array_equal(to_np(cs), cr)


@pytest.mark.parametrize("io,B,D,H", [("f32", 5, 64, 2), ("bf16", 19, 256, 2), ("bf16", 33, 600, 2)])
def test_decode_chain_equals_oracle_prefill(oracle, io, B, D, H):
    import torch
    from paper_2402_19427_b200 import binding
    T0, steps = 6, 9
    inp = synth.make_inputs(B, T0 + steps, D, H, io=io, seed=11, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], io)
    x = to_dev(inp["x"], io)
    _, h, cs = binding.prefill(x[:, :T0].contiguous(), params, flags=GENERIC)
    ys = []
    for t in range(T0, T0 + steps):
        ys.append(binding.decode_step(x[:, t].contiguous(), params, h, cs, flags=GENERIC))
    torch.cuda.synchronize()
    yr, hr, cr = oracle_prefill(oracle, inp)
    assert_close("y", np.stack([to_np(v) for v in ys], 1), yr[:, T0:], io)
    assert_close("h", to_np(h), hr, io)
    assert np.array_equal(to_np(cs), cr)                 # shifted raw inputs: bit-exact


def run_backward(oracle, inp, with_state):
    import torch
    from paper_2402_19427_b200 import binding
    io = inp["io"]
    params = binding.Params.from_numpy(inp["params"], io)
    h0 = inp["h0"] if with_state else None
    cs = inp["conv_state"] if with_state else None
    g = binding.backward(to_dev(inp["x"], io), params, to_dev(inp["dy"], io), h0=to_dev(h0), conv_state_in=to_dev(cs, io),
                         flags=GENERIC)
    torch.cuda.synchronize()
    gr = oracle.backward(inp["x"].astype(np.float64), f64(inp["params"]), inp["H"], inp["dy"].astype(np.float64),
                         h0=None if h0 is None else h0.astype(np.float64), conv_state_in=None if cs is None else cs.astype(np.float64))
    return {k: to_np(v) for k, v in g.items()}, gr


def test_backward_tiny_fp32_matches_oracle_and_finite_differences(oracle):
    """The T=64, D=64 gradient check: GPU fp32 backward == oracle analytic backward (itself pinned by central
    differences), and a directional central difference of the oracle forward agrees with the GPU gradient."""
    inp = synth.make_inputs(2, 64, 64, 2, io="f32", seed=4, with_dy=True, with_state=True, bias_scale=0.2)
    g, gr = run_backward(oracle, inp, with_state=True)
    for k in gr:
        scale = max(1.0, float(np.abs(gr[k]).max()))
        assert_close("d" + k, g[k], gr[k], "f32", scale=scale)
    rng = np.random.default_rng(5)
    p = f64(inp["params"]); x = inp["x"].astype(np.float64); dy = inp["dy"].astype(np.float64)
    h0 = inp["h0"].astype(np.float64); cs = inp["conv_state"].astype(np.float64)
    dirs = {k: rng.normal(size=v.shape) for k, v in p.items()}; dx = rng.normal(size=x.shape)
    eps = 1e-6
    def L(s):
        y, _, _ = oracle.prefill(x + s * dx, {k: v + s * dirs[k] for k, v in p.items()}, inp["H"], h0=h0, conv_state_in=cs)
        return float(np.sum(dy * y))
    num = (L(eps) - L(-eps)) / (2 * eps)
    ana = float(np.sum(g["x"] * dx) + sum(np.sum(g[k] * dirs[k]) for k in p))
    assert abs(num - ana) <= 2e-4 * max(1.0, abs(num))


@pytest.mark.parametrize("B,T,D,H,io", [(1, 5, 8, 2, "f32"), (2, 70, 600, 2, "f32"), (3, 129, 128, 4, "bf16")])
def test_backward_shapes(oracle, B, T, D, H, io):
    inp = synth.make_inputs(B, T, D, H, io=io, seed=31 + T, with_dy=True, with_state=True, bias_scale=0.2)
    g, gr = run_backward(oracle, inp, with_state=(T != 5))
    for k in gr:
        scale = max(1.0, float(np.abs(gr[k]).max())) if io == "f32" else 1.0
        assert_close("d" + k, g[k], gr[k], io, scale=scale)


def test_status_word_reads_ok_on_fresh_workspace():
    import torch
    from paper_2402_19427_b200 import binding
    ws = torch.randint(0, 255, (4096,), dtype=torch.uint8, device="cuda")
    assert binding.query_status(ws) == binding.OK


def test_recorded_timeout_is_reported_once_and_wait_limit_knob_round_trips():
    """Host side of the failure path: a status word as a kernel leaves it after a wait ran out (magic | code) is reported
    by rglru_query_status and cleared; the wait limit can be changed and restored.  No wait is made to run out here."""
    import torch
    from paper_2402_19427_b200 import binding
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    ws[:4] = torch.tensor([binding.ERR_TIMEOUT, 0x4C, 0x47, 0x52], dtype=torch.uint8)   # 0x52474C00 | 7, little endian
    assert binding.query_status(ws) == binding.ERR_TIMEOUT
    assert binding.query_status(ws) == binding.OK
    prev = binding.set_wait_limit_ns(123456789)
    assert prev == 2_000_000_000
    assert binding.set_wait_limit_ns(0) == 123456789
    assert binding.set_wait_limit_ns(0) == 2_000_000_000


@pytest.mark.parametrize("B,T,D,H,io,flags", [(2, 33, 32, 2, "f32", 1), (1, 2, 16, 2, "f32", 1), (2, 1, 8, 1, "f32", 1),
                                               (2, 64, 512, 2, "bf16", 0), (1, 200, 256, 1, "bf16", 0), (2, 70, 256, 2, "bf16", 1)])
def test_backward_through_the_carried_state(oracle, B, T, D, H, io, flags):
    """dh0 and d conv_state_in, with gradient arriving on h_T and conv_state_out, against the oracle: CUDA-core kernels
    (fp32, and bf16 forced generic) and the tensor-core backward (bf16, head width 256, T a multiple of 8)."""
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(B, T, D, H, io=io, seed=71 + T, with_dy=True, with_state=True, bias_scale=0.2)
    rng = np.random.default_rng(5)
    dhT = rng.normal(size=(B, D)).astype(np.float32)
    dcs = rng.normal(size=(B, 3, D)).astype(np.float32)
    if io == "bf16":
        dcs = synth.round_to_bf16(dcs)
    params = binding.Params.from_numpy(inp["params"], io)
    g = binding.backward(to_dev(inp["x"], io), params, to_dev(inp["dy"], io), h0=to_dev(inp["h0"]),
                         conv_state_in=to_dev(inp["conv_state"], io), flags=flags, dh_T=to_dev(dhT), dconv_state_out=to_dev(dcs, io),
                         state_grads=True)
    torch.cuda.synchronize()
    gr = oracle.backward(inp["x"].astype(np.float64), f64(inp["params"]), H, inp["dy"].astype(np.float64), h0=inp["h0"].astype(np.float64),
                         conv_state_in=inp["conv_state"].astype(np.float64), dh_T=dhT.astype(np.float64),
                         dconv_state_out=dcs.astype(np.float64), state_grads=True)
    for k in gr:
        scale = max(1.0, float(np.abs(gr[k]).max())) if io == "f32" else 1.0
        assert_close("d" + k, to_np(g[k]), gr[k], io, scale=scale)


def test_backward_of_two_chained_segments_on_the_gpu_matches_the_whole(oracle):
    """Truncated segments compose on the GPU as they do in the oracle: last segment first, its dh0 / d conv_state_in fed to
    the segment before it.  Compared with the oracle's backward of the whole sequence."""
    import torch
    from paper_2402_19427_b200 import binding
    B, T1, T2, D, H = 2, 128, 72, 256, 1
    inp = synth.make_inputs(B, T1 + T2, D, H, io="bf16", seed=88, with_dy=True, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); dy = to_dev(inp["dy"], "bf16")
    x1, x2 = x[:, :T1].contiguous(), x[:, T1:].contiguous()
    h0 = to_dev(inp["h0"]); cs0 = to_dev(inp["conv_state"], "bf16")
    y1, h1, cs1 = binding.prefill(x1, params, h0=h0, conv_state_in=cs0)
    g2 = binding.backward(x2, params, dy[:, T1:].contiguous(), h0=h1, conv_state_in=cs1, state_grads=True)
    g1 = binding.backward(x1, params, dy[:, :T1].contiguous(), h0=h0, conv_state_in=cs0, y=y1, dh_T=g2["h0"],
                          dconv_state_out=g2["conv_state"], state_grads=True)
    torch.cuda.synchronize()
    gr = oracle.backward(inp["x"].astype(np.float64), f64(inp["params"]), H, inp["dy"].astype(np.float64), h0=inp["h0"].astype(np.float64),
                         conv_state_in=inp["conv_state"].astype(np.float64), state_grads=True)
    assert_close("dx", np.concatenate([to_np(g1["x"]), to_np(g2["x"])], 1), gr["x"], "bf16")
    for k in ("conv_w", "conv_b", "W_a", "b_a", "W_x", "b_x", "lam"):
        assert_close("d" + k, to_np(g1[k]) + to_np(g2[k]), gr[k], "bf16")
    assert_close("dh0", to_np(g1["h0"]), gr["h0"], "bf16")
    assert_close("dconv_state", to_np(g1["conv_state"]), gr["conv_state"], "bf16")
