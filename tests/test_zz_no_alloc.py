"""rglru_prefill_static_scratch: the prefill for callers that cannot allocate device memory.

A serving process that froze its memory pool at start-up (or runs under an allocator that forbids side
allocations) cannot hand the library a workspace.  The entry point under test keeps the kernel's scratch in
an array inside the library instead.  Here it is called through the C ABI twice in a row, on different
inputs, and each result is compared with the regular entry point's (same kernel, caller-provided workspace) and with
the fp64 oracle.  The second call finds the first call's records still in the shared array and must not be confused
by them.  A third call updates the state in place (h_T over h0, conv_state_out over conv_state_in), which goes through
the private copies the entry point keeps in the same array.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

from paper_2402_19427_b200 import inputs as synth
from util import assert_close, oracle_prefill, to_dev, to_np

pytestmark = pytest.mark.gpu


def _run_both(binding, torch, inp):
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    h0 = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")
    B, T, D = x.shape
    # every buffer the no-allocation call touches is provided by the caller, outputs included
    y = torch.empty_like(x)
    hT = torch.empty(B, D, dtype=torch.float32, device=x.device)
    cso = torch.empty(B, 3, D, dtype=torch.bfloat16, device=x.device)
    status = torch.zeros(1, dtype=torch.int32, device=x.device)
    binding.prefill_static_scratch(x, params, y, hT, cso, h0=h0, conv_state_in=cs, status_word=status)
    assert binding.query_status(status) == binding.OK
    yr, hr, cr = binding.prefill(x, params, h0=h0, conv_state_in=cs)
    torch.cuda.synchronize()
    return (to_np(y), to_np(hT), to_np(cso)), (to_np(yr), to_np(hr), to_np(cr))


def test_static_scratch_prefill_matches_regular_prefill_twice(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    # 1st call: 2 sequences x 700 tokens x 2 heads -> 6 tiles per sequence, time split across CTAs
    # 2nd call: another shape and seed, so stale records of the first call sit where the second one looks
    for seed, (B, T, H) in ((41, (2, 700, 2)), (42, (3, 1000, 1))):
        inp = synth.make_inputs(B, T, 256 * H, H, io="bf16", seed=seed, with_state=True, bias_scale=0.3)
        got, ref = _run_both(binding, torch, inp)
        assert_close("y", got[0], ref[0], "bf16")
        assert_close("h_T", got[1], ref[1], "bf16")
        assert np.array_equal(got[2], ref[2])
        # the sibling call runs the same kernel; the oracle does not
        yo, ho, co = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
        assert_close("y vs oracle", got[0], yo, "bf16")
        assert_close("h_T vs oracle", got[1], ho, "bf16")
        assert np.array_equal(got[2], co)
        # how much of the tolerance's rms floor is in play: fraction of entries within the pure relative bound
        rel_ok = float(np.mean(np.abs(got[0] - yo) <= 2e-2 * np.abs(yo)))
        assert rel_ok > 0.97, rel_ok


def test_static_scratch_prefill_with_state_updated_in_place(oracle):
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(2, 700, 512, 2, io="bf16", seed=43, with_state=True, bias_scale=0.3)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    x = to_dev(inp["x"], "bf16")
    h = to_dev(inp["h0"]); cs = to_dev(inp["conv_state"], "bf16")      # state in, overwritten by state out
    y = torch.empty_like(x)
    status = torch.zeros(1, dtype=torch.int32, device=x.device)
    binding.prefill_static_scratch(x, params, y, h, cs, h0=h, conv_state_in=cs, status_word=status)
    assert binding.query_status(status) == binding.OK
    yr, hr, cr = binding.prefill(x, params, h0=to_dev(inp["h0"]), conv_state_in=to_dev(inp["conv_state"], "bf16"))
    torch.cuda.synchronize()
    assert_close("y", to_np(y), to_np(yr), "bf16"); assert_close("h_T", to_np(h), to_np(hr), "bf16")
    assert np.array_equal(to_np(cs), to_np(cr))
    yo, ho, co = oracle_prefill(oracle, inp, h0=inp["h0"].astype(np.float64), cs=inp["conv_state"].astype(np.float64))
    assert_close("y vs oracle", to_np(y), yo, "bf16"); assert_close("h_T vs oracle", to_np(h), ho, "bf16")
    assert np.array_equal(to_np(cs), co)


def test_static_scratch_rejects_what_it_cannot_serve():
    import torch
    from paper_2402_19427_b200 import binding
    inp = synth.make_inputs(1, 8, 256, 1, io="bf16", seed=5)
    params = binding.Params.from_numpy(inp["params"], "bf16")
    dev = params.conv_w.device
    # scratch for 64 x 4096 tokens of 16 heads is far beyond the 8 MiB array: refused on the host, nothing runs
    big = binding.make_shape(64, 4096, 4096, 16, torch.bfloat16)
    assert 256 + binding.workspace_bytes(big, binding.OP_PREFILL) > binding.STATIC_SCRATCH_BYTES
    lib = binding.load()
    import ctypes
    good = ctypes.c_void_p(params.conv_w.data_ptr())
    p16 = binding.Params.from_numpy(synth.make_inputs(1, 4, 4096, 16, io="bf16", seed=6)["params"], "bf16")
    rc = lib.rglru_prefill_static_scratch(ctypes.byref(big), ctypes.byref(p16.ptrs), good, None, None,
                                          ctypes.c_void_p(params.W_a.data_ptr()), good, good, None, None)
    assert rc == binding.ERR_WORKSPACE
    # fp32 io has no tensor-core kernel and therefore no scratch-using variant
    f32 = binding.make_shape(1, 8, 256, 1, torch.float32)
    rc = lib.rglru_prefill_static_scratch(ctypes.byref(f32), ctypes.byref(params.ptrs), good, None, None,
                                          ctypes.c_void_p(params.W_a.data_ptr()), good, good, None, None)
    assert rc == binding.ERR_UNSUPPORTED
    assert dev.type == "cuda"
