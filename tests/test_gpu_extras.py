"""GPU parity of the optional extras of the forward (rglru_prefill_ex) against the fp64 oracle, on the CUDA-core kernels
(fp32 and bf16, any head width) and on the tensor-core kernel (bf16, head width 256): the merged output of the recurrent
block, y_t = h_t * GeLU(branch_t) (Section 2.3), and the decay product of the call, prod_t a_t, which together with h_T from
a zero state describes the call as one affine step of Eq. 4."""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import assert_close, f64, to_dev, to_np

pytestmark = pytest.mark.gpu


def run_both(oracle, B, T, D, H, io, seed, flags=0, with_state=True):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(B, T, D, H, io=io, seed=seed, with_state=with_state, bias_scale=0.3)
    rng = np.random.default_rng(seed + 1)
    branch = (rng.standard_normal((B, T, D)) * 1.5).astype(np.float32)
    if io == "bf16":
        branch = synth.round_to_bf16(branch)
    params = binding.Params.from_numpy(inp["params"], io)
    h0 = inp["h0"] if with_state else None
    cs = inp["conv_state"] if with_state else None
    a_prod = torch.full((B, D), -7.0, dtype=torch.float32, device="cuda")
    y, hT, cso = binding.prefill(to_dev(inp["x"], io), params, h0=None if h0 is None else to_dev(h0),
                                 conv_state_in=None if cs is None else to_dev(cs, io), flags=flags,
                                 gate_branch=to_dev(branch, io), a_prod=a_prod)
    torch.cuda.synchronize()
    yr, hr, cr, ar = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), H, c=inp["c"],
                                    h0=None if h0 is None else h0.astype(np.float64),
                                    conv_state_in=None if cs is None else cs.astype(np.float64),
                                    gate_branch=branch.astype(np.float64), with_a_prod=True)
    assert_close("y", to_np(y), yr, io); assert_close("h_T", to_np(hT), hr, io)
    assert np.array_equal(to_np(cso), cr)
    return to_np(a_prod), ar, inp, params


def check_product(got, ref, io):
    """prod_t a_t lies in (0, 1) and may be tiny; it is compared in the log domain: log prod = sum_t log a_t, T terms each
    within the gate tolerance of the path."""
    assert np.all(got >= 0) and np.all(got <= 1)
    big = ref > 1e-30
    tol = 2e-2 if io == "bf16" else 1e-4
    np.testing.assert_allclose(np.log(got[big]), np.log(ref[big]), rtol=tol, atol=tol)
    assert np.all(got[~big] < 1e-25)


@pytest.mark.parametrize("io,B,T,D,H", [("f32", 2, 37, 64, 2), ("f32", 1, 130, 96, 3), ("bf16", 2, 70, 128, 4)])
def test_extras_on_the_cuda_core_kernels(oracle, io, B, T, D, H):
    got, ref, _, _ = run_both(oracle, B, T, D, H, io, seed=600 + T)
    check_product(got, ref, io)


@pytest.mark.parametrize("B,T,H", [(1, 1, 1), (2, 65, 1), (1, 129, 2), (3, 320, 1), (1, 1000, 1), (9, 200, 2)])
def test_extras_on_the_tensor_core_kernel(oracle, B, T, H):
    """(9, 200, 2): nine sequences over the pairs of a head, so some are dealt whole and one is split in time (look-back)."""
    import torch
    from paper_2402_19427_b200 import binding
    D = 256 * H
    assert binding.workspace_bytes(binding.make_shape(B, T, D, H, torch.bfloat16), binding.OP_PREFILL) > 256
    got, ref, _, _ = run_both(oracle, B, T, D, H, "bf16", seed=700 + T)
    check_product(got, ref, "bf16")


def test_one_long_sequence_split_over_all_pairs(oracle):
    """B = 1: every tile takes its incoming state, and the running product, from the look-back."""
    got, ref, _, _ = run_both(oracle, 1, 4096, 256, 1, "bf16", seed=91, with_state=False)
    check_product(got, ref, "bf16")


def test_call_as_one_affine_step_on_the_gpu(oracle):
    """h_T(h0) = a_prod * h0 + h_T(0) with both runs on the GPU; and two time shares chained through (a_prod, h_T from
    zero) reproduce the state of the whole (what ranks that split a sequence in time exchange)."""
    import torch
    from paper_2402_19427_b200 import binding, sharding
    B, T, D, H = 2, 300, 512, 2
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=17, with_state=True)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16"); h0 = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    ap = torch.empty(B, D, dtype=torch.float32, device="cuda")
    _, hz, _ = binding.prefill(x, params, conv_state_in=cs, a_prod=ap)
    _, h1, _ = binding.prefill(x, params, h0=h0, conv_state_in=cs)
    torch.cuda.synchronize()
    ref = ap * h0 + hz
    assert float((h1 - ref).abs().max()) <= 1e-4 * float(h1.abs().max())
    T1 = 160
    a1 = torch.empty_like(ap); a2 = torch.empty_like(ap)
    _, b1, c1 = binding.prefill(x[:, :T1].contiguous(), params, conv_state_in=cs, a_prod=a1)
    _, b2, _ = binding.prefill(x[:, T1:].contiguous(), params, conv_state_in=c1, a_prod=a2)
    A, Bv = sharding.combine_steps((a1, b1), (a2, b2))
    torch.cuda.synchronize()
    assert float((A * h0 + Bv - h1).abs().max()) <= 1e-4 * float(h1.abs().max())
    _, hr, _ = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), H, h0=inp["h0"].astype(np.float64),
                              conv_state_in=inp["conv_state"].astype(np.float64))
    assert_close("h_T", to_np(A * h0 + Bv), hr, "bf16")


class _ThreadRanks:
    """Stand-in for torch.distributed inside one process: every "rank" is a host thread, an all-gather is a hand-over through
    a shared list between two host barriers.  Only the host side waits; the ranks' kernels are independent launches."""

    def __init__(self, world):
        import threading
        self.world, self.slots, self.barrier, self.local = world, [None] * world, threading.Barrier(world), threading.local()

    def get_rank(self):
        return self.local.rank

    def get_world_size(self):
        return self.world

    def all_gather(self, out_list, tensor):
        import torch
        torch.cuda.synchronize()
        self.slots[self.local.rank] = tensor
        self.barrier.wait()
        for i in range(self.world):
            out_list[i].copy_(self.slots[i])
        torch.cuda.synchronize()
        self.barrier.wait()


@pytest.mark.parametrize("world,with_state", [(2, True), (3, False)])
def test_time_shares_on_the_gpu_equal_the_uncut_prefill(oracle, world, with_state):
    """sharding.prefill_time_share, the GPU path of a prefill cut along time, run by `world` host threads that stand for the
    ranks (one GPU here): Conv1D history and affine steps are exchanged, every share is then computed from its true incoming
    state, and the concatenation matches the oracle's uncut prefill; the last share ends in the final state."""
    import threading
    import torch
    from paper_2402_19427_b200 import binding, sharding
    B, T, D, H = 2, 450, 512, 2
    inp = synth.make_inputs(B, T, D, H, io="bf16", seed=41, with_state=True, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    h0 = to_dev(inp["h0"]) if with_state else None
    cs = to_dev(inp["conv_state"], "bf16") if with_state else None
    ranks = _ThreadRanks(world)
    out, errs = [None] * world, []

    def run(r):
        try:
            ranks.local.rank = r
            torch.cuda.set_device(0)
            t0, tc = sharding.split_range(T, world, r)
            out[r] = sharding.prefill_time_share(x[:, t0:t0 + tc].contiguous(), params, ranks, h0=h0, conv_state_in=cs)
            torch.cuda.synchronize()
        except Exception as e:   # noqa: BLE001
            errs.append(e)
            ranks.barrier.abort()

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errs, errs
    yr, hr, cr = oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), H, c=inp["c"],
                                h0=inp["h0"].astype(np.float64) if with_state else None,
                                conv_state_in=inp["conv_state"].astype(np.float64) if with_state else None)
    assert_close("y", np.concatenate([to_np(o[0]) for o in out], 1), yr, "bf16")
    assert_close("h_T", to_np(out[-1][1]), hr, "bf16")
    assert np.array_equal(to_np(out[-1][2]), cr)
