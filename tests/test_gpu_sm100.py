"""GPU parity of the tcgen05 fused prefill (bf16 io, head width 256) against the fp64 oracle, through the C ABI.
Covers ragged tails, T < 3, incoming state, several heads, the cross-CTA carry of the time split, long-memory
channels, channels outside the polynomial-exp range, and sampled heads of the full-size workloads."""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import Guarded, assert_close, f64, gpu_prefill, oracle_prefill, to_dev, to_np

pytestmark = pytest.mark.gpu


def uses_sm100(B, T, D, H):
    from paper_2402_19427_b200 import binding
    import torch
    return binding.workspace_bytes(binding.make_shape(B, T, D, H, torch.bfloat16), binding.OP_PREFILL) > 256


@pytest.mark.parametrize("B,T,H", [(1, 1, 1), (2, 2, 1), (1, 3, 2), (1, 31, 1), (2, 64, 1), (1, 65, 1), (1, 128, 2), (3, 129, 1),
                                   (2, 320, 2), (1, 1000, 1), (5, 257, 3)])
def test_shapes_with_state_and_bias(oracle, B, T, H):
    D = 256 * H
    assert uses_sm100(B, T, D, H)
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=500 + T, with_state=True, bias_scale=0.5)
    y, hT, cso = gpu_prefill(inp, h0=inp["h0"], cs=inp["conv_state"])
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")
    assert np.array_equal(cso, cr)


def test_more_half_heads_than_sms_runs_in_waves(oracle):
    """80 heads = 160 half-head CTAs on 148 SMs: no time split, an ordinary launch whose CTAs run in two waves."""
    B, T, H = 2, 130, 80
    D = 256 * H
    assert uses_sm100(B, T, D, H)
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=77, with_state=True, bias_scale=0.5)
    y, hT, cso = gpu_prefill(inp, h0=inp["h0"], cs=inp["conv_state"])
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")
    assert np.array_equal(cso, cr)


def test_zero_state_defaults_and_generic_agreement(oracle):
    inp = synth.make_inputs(2, 200, 512, 2, io="bf16", seed=3)
    y, hT, cso = gpu_prefill(inp)
    yg, hg, cg = gpu_prefill(inp, flags=1)
    yr, hr, cr = oracle_prefill(oracle, inp)
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")
    assert_close("y generic", yg, yr, "bf16")
    assert np.array_equal(cso, cr) and np.array_equal(cg, cr)


def test_long_sequence_cross_cta_carry_and_long_memory(oracle):
    """One sequence of 40 tiles on two half-head groups: every tile's state arrives through the look-back;
    5 % of the channels have a^c = 0.9999 so the carry matters over thousands of tokens."""
    inp = synth.make_inputs(1, 5000, 256, 1, io="bf16", seed=9, long_memory_frac=0.05, with_state=True)
    y, hT, cso = gpu_prefill(inp, h0=inp["h0"], cs=inp["conv_state"])
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")
    assert np.array_equal(cso, cr)


def test_wide_lambda_range_uses_exp_path(oracle):
    """Lambda down to -3 (a = 0.047): decay rates far outside the polynomial range; and up to 16 (a^c ~ 1 - 1e-6)."""
    inp = synth.make_inputs(2, 300, 256, 1, io="bf16", seed=21, bias_scale=0.3)
    rng = np.random.default_rng(1)
    inp["params"]["lam"] = rng.uniform(-3.0, 16.0, size=256).astype(np.float32)
    y, hT, _ = gpu_prefill(inp)
    yr, hr, _ = oracle_prefill(oracle, inp)
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")


def test_split_prefill_and_aliased_state(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(2, 700, 512, 2, io="bf16", seed=17, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    h = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    y1, _, _ = binding.prefill(x[:, :2].contiguous(), params, h0=h, conv_state_in=cs, h_T=h, conv_state_out=cs)
    y2, _, _ = binding.prefill(x[:, 2:301].contiguous(), params, h0=h, conv_state_in=cs, h_T=h, conv_state_out=cs)
    y3, _, _ = binding.prefill(x[:, 301:].contiguous(), params, h0=h, conv_state_in=cs, h_T=h, conv_state_out=cs)
    torch.cuda.synchronize()
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", np.concatenate([to_np(y1), to_np(y2), to_np(y3)], 1), yr, "bf16")
    assert_close("h_T", to_np(h), hr, "bf16")
    assert np.array_equal(to_np(cs), cr)


def test_status_ok_and_repeatable():
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(1, 2000, 512, 2, io="bf16", seed=2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    shape = binding.make_shape(1, 2000, 512, 2, torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, x.device)
    outs = []
    for _ in range(3):
        y, hT, _ = binding.prefill(x, params, workspace=ws)
        outs.append((y.clone(), hT.clone()))
    assert binding.query_status(ws) == binding.OK
    for y, hT in outs[1:]:
        assert torch.equal(y, outs[0][0]) and torch.equal(hT, outs[0][1])   # same reduction order every run


@pytest.mark.parametrize("B,H,T0,steps", [(1, 1, 4, 5), (19, 1, 6, 9), (130, 2, 3, 4), (77, 3, 1, 3), (300, 1, 2, 2)])
def test_decode_chain_equals_oracle_prefill(oracle, B, H, T0, steps):
    """Tensor-core decode step (cluster pair per head and batch tile): prefill of T0 tokens, then chained
    single-token steps; outputs, final h and the shifted conv state against the oracle's prefill of T0 + steps."""
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    inp = synth.make_inputs(B, T0 + steps, D, H, io="bf16", seed=700 + B, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    _, h, cs = binding.prefill(x[:, :T0].contiguous(), params)
    ys = [binding.decode_step(x[:, t].contiguous(), params, h, cs) for t in range(T0, T0 + steps)]
    torch.cuda.synchronize()
    yr, hr, cr = oracle_prefill(oracle, inp)
    assert_close("y", np.stack([to_np(v) for v in ys], 1), yr[:, T0:], "bf16")
    assert_close("h", to_np(h), hr, "bf16")
    assert np.array_equal(to_np(cs), cr)


def test_decode_agrees_with_generic_decode_and_status():
    import torch
    from paper_2402_19427_b200 import binding
    B, H = 48, 2
    inp = synth.make_inputs(B, 4, 256 * H, H, io="bf16", seed=33, with_state=True, bias_scale=0.2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    outs = []
    for flags in (0, 1):
        h = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
        ws = binding.alloc_workspace(binding.make_shape(B, 1, 256 * H, H, torch.bfloat16), binding.OP_DECODE, x.device)
        ys = [binding.decode_step(x[:, t].contiguous(), params, h, cs, flags=flags, workspace=ws) for t in range(4)]
        assert binding.query_status(ws) == binding.OK
        outs.append((torch.stack(ys, 1), h, cs))
    assert_close("y", to_np(outs[0][0]), to_np(outs[1][0]), "bf16")
    assert_close("h", to_np(outs[0][1]), to_np(outs[1][1]), "bf16")
    assert torch.equal(outs[0][2], outs[1][2])


@pytest.mark.parametrize("B,T,H,with_y", [(3, 8, 1, True), (2, 136, 1, True), (1, 264, 2, False), (2, 1000, 1, True)])
def test_backward_tensor_core_path(oracle, B, T, H, with_y):
    """Tensor-core backward (GEMMs for z, du and dW around the chunked reverse scan) against the oracle's analytic
    gradients; with and without the saved forward output."""
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=900 + T, with_dy=True, with_state=True, bias_scale=0.2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); dy = to_dev(inp["dy"], "bf16")
    h0 = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    shape = binding.make_shape(B, T, D, H, torch.bfloat16)
    assert binding.workspace_bytes(shape, binding.OP_BACKWARD) != binding.workspace_bytes(
        binding.make_shape(B, T, D, H, torch.bfloat16, flags=1), binding.OP_BACKWARD)      # not the generic path
    y = binding.prefill(x, params, h0=h0, conv_state_in=cs)[0] if with_y else None
    ws = binding.alloc_workspace(shape, binding.OP_BACKWARD, x.device)
    g = binding.backward(x, params, dy, h0=h0, conv_state_in=cs, y=y, workspace=ws)
    assert binding.query_status(ws) == binding.OK
    gr = oracle.backward(inp["x"].astype(np.float64), f64(inp["params"]), H, inp["dy"].astype(np.float64),
                         h0=inp["h0"].astype(np.float64), conv_state_in=inp["conv_state"].astype(np.float64))
    for k in gr:
        assert_close("d" + k, to_np(g[k]), gr[k], "bf16")


def test_backward_is_run_to_run_identical():
    """Every parameter gradient is a sum over B*T tokens taken in a fixed order (per-chunk partial sums, then one reduction
    over the chunks; no atomics), so two runs on the same inputs agree bit for bit; so do dx and the prefill outputs."""
    import torch
    from paper_2402_19427_b200 import binding
    B, T, H = 3, 520, 2
    D = 256 * H
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=31, with_dy=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); dy = to_dev(inp["dy"], "bf16")
    shape = binding.make_shape(B, T, D, H, torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_BACKWARD, x.device)
    runs = []
    for _ in range(2):
        y = binding.prefill(x, params)[0]
        g = binding.backward(x, params, dy, y=y, workspace=ws)
        torch.cuda.synchronize()
        runs.append({k: to_np(v).copy() for k, v in g.items()} | {"y": to_np(y).copy()})
    for k in runs[0]:
        assert np.array_equal(runs[0][k], runs[1][k]), k


@pytest.mark.parametrize("B,T,H", [(5, 300, 2), (2, 1300, 1), (40, 20, 1)])
def test_prefill_host_pipelined_chunks_match_device_prefill(oracle, B, T, H):
    """rglru_prefill_host cuts the batch into chunks of whole sequences (one each, or several when there are more
    sequences than chunks) that are copied in, run and copied out concurrently; the result must be the forward of the
    whole batch."""
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=77, with_state=True, bias_scale=0.2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    h0 = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    x_pin = torch.from_numpy(inp["x"]).to(torch.bfloat16).pin_memory()
    y_pin = torch.empty(B, T, D, dtype=torch.bfloat16).pin_memory()
    hT_pin = torch.empty(B, D, dtype=torch.float32).pin_memory()
    cs_pin = torch.empty(B, 3, D, dtype=torch.bfloat16).pin_memory()
    shape = binding.make_shape(B, T, D, H, torch.bfloat16)
    ws = binding.alloc_workspace(shape, binding.OP_PREFILL, h0.device)
    staging = torch.empty(binding.host_staging_bytes(shape), dtype=torch.uint8, device=h0.device)
    for _ in range(2):   # twice: the helper streams and events are reused
        binding.prefill_host(x_pin, params, y_pin, hT_pin, cs_pin, staging, ws, h0=h0, conv_state_in=cs)
        torch.cuda.synchronize()
        assert binding.query_status(ws) == binding.OK
        yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
        assert_close("y", to_np(y_pin), yr, "bf16"); assert_close("h_T", to_np(hT_pin), hr, "bf16")
        assert np.array_equal(to_np(cs_pin), cr)
        y_pin.zero_()


@pytest.mark.parametrize("Dh,B,T,H", [(128, 2, 130, 2), (128, 3, 257, 4), (64, 2, 130, 4), (64, 1, 1000, 8), (128, 9, 200, 2)])
def test_narrower_heads_on_the_tensor_core_path(oracle, Dh, B, T, H):
    """Heads of width 128 and 64 (the 16 blocks of Section 4.1 at smaller D_RNN) run on the same kernel as
    groups of two or four heads whose block-diagonal weights fill a 256 x 256 block; a workspace larger than the bare
    status header shows that the tensor-core path was chosen.  The last case splits a sequence in time."""
    D = Dh * H
    assert D % 256 == 0 and uses_sm100(B, T, D, H)
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=800 + Dh + T, with_state=True, bias_scale=0.5)
    y, hT, cso = gpu_prefill(inp, h0=inp["h0"], cs=inp["conv_state"])
    yr, hr, cr = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y", y, yr, "bf16"); assert_close("h_T", hT, hr, "bf16")
    assert np.array_equal(cso, cr)
    # heads stay independent: changing one head's weights changes only that head's channels
    inp2 = {**inp, "params": dict(inp["params"])}
    W = inp2["params"]["W_a"].copy(); W[1] = -W[1]; inp2["params"]["W_a"] = W
    y2, _, _ = gpu_prefill(inp2, h0=inp["h0"], cs=inp["conv_state"])
    other = np.ones(D, bool); other[Dh:2 * Dh] = False
    assert np.array_equal(y2[:, :, other], y[:, :, other]) and not np.array_equal(y2[:, :, ~other], y[:, :, ~other])


@pytest.mark.parametrize("Dh,B,H,T0,steps", [(128, 19, 2, 5, 6), (128, 130, 4, 3, 4), (64, 33, 4, 4, 5), (64, 200, 8, 2, 3),
                                                 (160, 19, 2, 5, 6), (96, 130, 3, 3, 4), (160, 70, 16, 2, 3), (224, 5, 1, 4, 4), (128, 40, 3, 3, 3)])
def test_decode_chain_with_narrower_heads(oracle, Dh, B, H, T0, steps):
    """Decode steps for heads narrower than 256 on the tensor-core kernel: widths 128 and 64 as groups of two or four heads per
    256 channels (a CTA then needs only the channels it convolves itself), other multiples of 32 one head per 256 channel
    slots.  Checked against the oracle; the CUDA-core kernel, forced by flag, must agree within tolerance but not bit for bit,
    which shows that a different kernel ran by default."""
    import torch
    from paper_2402_19427_b200 import binding
    D = Dh * H
    inp = synth.make_inputs(B, T0 + steps, D, H, io="bf16", seed=900 + Dh + B, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    _, h0, cs0 = binding.prefill(x[:, :T0].contiguous(), params)
    outs = []
    for flags in (0, 1):
        h, cs = h0.clone(), cs0.clone()
        ys = [binding.decode_step(x[:, t].contiguous(), params, h, cs, flags=flags) for t in range(T0, T0 + steps)]
        outs.append((torch.stack(ys, 1), h, cs))
    torch.cuda.synchronize()
    yr, hr, cr = oracle_prefill(oracle, inp)
    for y, h, cs in outs:
        assert_close("y", to_np(y), yr[:, T0:], "bf16"); assert_close("h", to_np(h), hr, "bf16")
        assert np.array_equal(to_np(cs), cr)
    assert not torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("Dh,B,T,H,with_y", [(128, 2, 136, 2, True), (128, 1, 264, 4, False), (64, 2, 200, 4, True), (64, 1, 72, 8, False),
                                                 (160, 2, 136, 2, True), (96, 1, 264, 3, False), (160, 1, 200, 16, True), (224, 2, 72, 1, True),
                                                 (32, 1, 136, 5, True), (128, 2, 72, 3, True)])
def test_backward_with_narrower_heads(oracle, Dh, B, T, H, with_y):
    """Tensor-core backward for heads narrower than 256 (any multiple of 32): the GEMMs run on groups of 256 channel slots with
    block-diagonal weights and only the diagonal blocks of the weight gradient are returned; widths that do not fill the
    256 slots, and a partial last group, leave slots that do not exist.  All gradients, the state gradients included,
    against the oracle's analytic ones."""
    import torch
    from paper_2402_19427_b200 import binding
    D = Dh * H
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=950 + Dh + T, with_dy=True, with_state=True, bias_scale=0.2)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); dy = to_dev(inp["dy"], "bf16")
    h0 = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    shape = binding.make_shape(B, T, D, H, torch.bfloat16)
    assert binding.workspace_bytes(shape, binding.OP_BACKWARD) != binding.workspace_bytes(
        binding.make_shape(B, T, D, H, torch.bfloat16, flags=1), binding.OP_BACKWARD)      # not the generic path
    y = binding.prefill(x, params, h0=h0, conv_state_in=cs)[0] if with_y else None
    ws = binding.alloc_workspace(shape, binding.OP_BACKWARD, x.device)
    rng = np.random.default_rng(3)
    dhT = rng.standard_normal((B, D)).astype(np.float32)
    g = binding.backward(x, params, dy, h0=h0, conv_state_in=cs, y=y, workspace=ws, dh_T=to_dev(dhT), state_grads=True)
    assert binding.query_status(ws) == binding.OK
    gr = oracle.backward(inp["x"].astype(np.float64), f64(inp["params"]), H, inp["dy"].astype(np.float64),
                         h0=inp["h0"].astype(np.float64), conv_state_in=inp["conv_state"].astype(np.float64),
                         dh_T=dhT.astype(np.float64), state_grads=True)
    assert set(gr) <= set(g)
    for k in gr:
        assert_close("d" + k, to_np(g[k]), gr[k], "bf16")


@pytest.mark.parametrize("Dh,B,T,H", [(160, 2, 130, 2), (96, 3, 257, 3), (192, 1, 1000, 1), (224, 2, 65, 2), (32, 2, 100, 5), (128, 2, 100, 3),
                                      (160, 2, 300, 16), (160, 9, 200, 2)])
def test_head_widths_that_do_not_divide_256(oracle, Dh, B, T, H):
    """Section 4.1 fixes 16 blocks, so the paper's layers have head widths such as 96 (D_RNN = 1536) and 160 (D_RNN = 2560,
    the sixth case).  Such a head runs alone in the kernel's 256 channel slots; the slots beyond its width have zero weights
    and taps and are never written.  With incoming state (the first slab is then assembled from row copies), biases, a
    sequence split in time (last case), and the channels next to the last head's end, which lie outside the tensors."""
    import torch
    from paper_2402_19427_b200 import binding
    D = Dh * H
    assert uses_sm100(B, T, D, H)
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=1000 + Dh + T, with_state=True, bias_scale=0.5)
    rng = np.random.default_rng(Dh)
    branch = synth.round_to_bf16((rng.standard_normal((B, T, D)) * 1.5).astype(np.float32))
    for with_branch in (False, True):
        g = Guarded()
        y = g.empty((B, T, D), torch.bfloat16); hT = g.empty((B, D), torch.float32); cso = g.empty((B, 3, D), torch.bfloat16)
        ap = g.empty((B, D), torch.float32)
        binding.prefill(to_dev(inp["x"], "bf16"), binding.Params.from_numpy(inp["params"], "bf16"), h0=to_dev(inp["h0"]),
                        conv_state_in=to_dev(inp["conv_state"], "bf16"), y=y, h_T=hT, conv_state_out=cso, a_prod=ap,
                        gate_branch=to_dev(branch, "bf16") if with_branch else None)
        g.check()
        yr, hr, cr, ar = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), H, c=inp["c"], h0=inp["h0"].astype(np.float64),
                                        conv_state_in=inp["conv_state"].astype(np.float64), with_a_prod=True,
                                        gate_branch=branch.astype(np.float64) if with_branch else None)
        assert_close("y", to_np(y), yr, "bf16"); assert_close("h_T", to_np(hT), hr, "bf16")
        assert np.array_equal(to_np(cso), cr)
        big = ar > 1e-30
        np.testing.assert_allclose(np.log(to_np(ap)[big]), np.log(ar[big]), rtol=2e-2, atol=2e-2)
