"""Helpers shared by the GPU parity tests: upload seeded inputs, run the CUDA path through the C ABI,
run the oracle on the same values, compare with the stated tolerances."""
import numpy as np

from paper_2402_19427_b200 import inputs as synth

# Tolerances.  fp32 io: max abs error 1e-4 on y and h_T.  bf16 io (fp32 state): element-wise
# |gpu - ref| <= 2e-2 * max(|ref|, rms(ref)) per output tensor (relative for large entries, floored at
# the tensor's rms for entries near zero).
FP32_ATOL = 1e-4
BF16_REL = 2e-2


def torch_dtype(io):
    import torch
    return torch.bfloat16 if io == "bf16" else torch.float32


def to_dev(a, io=None, device="cuda"):
    import torch
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if io is not None:
        t = t.to(torch_dtype(io))
    return t.to(device).contiguous()


def to_np(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def f64(p):
    return {k: (None if v is None else np.asarray(v, dtype=np.float64)) for k, v in p.items()}


def assert_close(name, got, ref, io, scale=1.0):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    err = np.abs(got - ref)
    if io == "f32":
        worst = err.max() if err.size else 0.0
        assert worst <= FP32_ATOL * scale, f"{name}: max abs err {worst:.3e} > {FP32_ATOL * scale:.1e}"
    else:
        rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
        bound = BF16_REL * scale * np.maximum(np.abs(ref), rms)
        bad = err > bound
        if bad.any():
            i = np.unravel_index(np.argmax(err - bound), err.shape)
            raise AssertionError(f"{name}: {bad.sum()} of {bad.size} outside 2e-2*max(|ref|, rms={rms:.3e}); "
                                 f"worst at {i}: got {got[i]:.6e} ref {ref[i]:.6e}")


def gpu_prefill(inp, flags=0, h0=None, cs=None):
    """Run rglru_prefill on the GPU for a workload dict; returns float64 numpy (y, h_T, conv_state_out)."""
    from paper_2402_19427_b200 import binding
    io = inp["io"]
    params = binding.Params.from_numpy(inp["params"], io)
    x = to_dev(inp["x"], io)
    y, hT, cso = binding.prefill(x, params, h0=to_dev(h0), conv_state_in=to_dev(cs, io), c=inp["c"], flags=flags)
    import torch
    torch.cuda.synchronize()
    return to_np(y), to_np(hT), to_np(cso)


def oracle_prefill(oracle, inp, h0=None, cs=None):
    return oracle.prefill(inp["x"].astype(np.float64), f64(inp["params"]), inp["H"], c=inp["c"], h0=h0, conv_state_in=cs)


class Guarded:
    """Output buffers carved out of a larger allocation with canary bytes before and after each: the device code builds
    addresses by hand (swizzled tiles, clipped tiled stores), and the memory checker is closed on this machine, so every call
    that writes an output is followed by a check that the bytes around it are untouched."""
    PAD = 4096   # bytes on each side; a multiple of every alignment the library asks for
    FILL = 0xA5

    def __init__(self, device="cuda"):
        self.device = device
        self.items = []

    def empty(self, shape, dtype):
        import torch
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        body = (n + 255) // 256 * 256
        raw = torch.full((self.PAD + body + self.PAD,), self.FILL, dtype=torch.uint8, device=self.device)
        view = raw[self.PAD:self.PAD + n].view(dtype).view(*shape)
        self.items.append((raw, n))
        return view

    def check(self):
        import torch
        torch.cuda.synchronize()
        for k, (raw, n) in enumerate(self.items):
            head, tail = raw[:self.PAD], raw[self.PAD + n:]
            assert bool((head == self.FILL).all()), f"guard bytes before output {k} were overwritten"
            assert bool((tail == self.FILL).all()), f"guard bytes after output {k} were overwritten"
