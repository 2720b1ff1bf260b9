"""Thin ctypes binding over the C ABI in ``include/rglru.h``.

Argument marshalling only: every step of the path (Conv1D, gates, decay, scan, state hand-off,
backward) runs inside the CUDA library.  PyTorch appears here for device memory and streams.
There is no fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librglru_b200.so")

OK, ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGN, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_ALIAS = range(9)
F32, BF16 = 0, 1
OP_PREFILL, OP_DECODE, OP_BACKWARD = 0, 1, 2
FLAG_NONE, FLAG_FORCE_GENERIC = 0, 1
FLAG_TEST_CARRY_NEVER_ARRIVES = 0x40000000   # failure-path test hook of the tensor-core prefill (see include/rglru.h)

EXPORTED = ["rglru_abi_version", "rglru_status_string", "rglru_workspace_bytes", "rglru_prefill",
            "rglru_decode_step", "rglru_backward", "rglru_host_staging_bytes", "rglru_prefill_host",
            "rglru_query_status", "rglru_prefill_static_scratch", "rglru_set_wait_limit_ns", "rglru_prefill_ex"]


class Shape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("D", ctypes.c_int32), ("H", ctypes.c_int32),
                ("io", ctypes.c_int32), ("c", ctypes.c_float), ("flags", ctypes.c_uint32)]


class ParamPtrs(ctypes.Structure):
    _fields_ = [("conv_w", ctypes.c_void_p), ("conv_b", ctypes.c_void_p), ("W_a", ctypes.c_void_p),
                ("b_a", ctypes.c_void_p), ("W_x", ctypes.c_void_p), ("b_x", ctypes.c_void_p),
                ("lam", ctypes.c_void_p)]


class RglruError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (``python -m paper_2402_19427_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2402_19427_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
        sp, pp = ctypes.POINTER(Shape), ctypes.POINTER(ParamPtrs)
        lib.rglru_abi_version.restype = i32
        lib.rglru_status_string.argtypes = [i32]
        lib.rglru_status_string.restype = ctypes.c_char_p
        lib.rglru_workspace_bytes.argtypes = [sp, i32]
        lib.rglru_workspace_bytes.restype = sz
        lib.rglru_prefill.argtypes = [sp, pp] + [vp] * 7 + [sz, vp]
        lib.rglru_prefill.restype = i32
        lib.rglru_prefill_ex.argtypes = [sp, pp] + [vp] * 8 + [sz, vp]
        lib.rglru_prefill_ex.restype = i32
        lib.rglru_decode_step.argtypes = [sp, pp] + [vp] * 5 + [sz, vp]
        lib.rglru_decode_step.restype = i32
        lib.rglru_backward.argtypes = [sp, pp] + [vp] * 15 + [sz, vp]
        lib.rglru_backward.restype = i32
        lib.rglru_host_staging_bytes.argtypes = [sp]
        lib.rglru_host_staging_bytes.restype = sz
        lib.rglru_prefill_host.argtypes = [sp, pp] + [vp] * 7 + [sz, vp, sz, vp]
        lib.rglru_prefill_host.restype = i32
        lib.rglru_prefill_static_scratch.argtypes = [sp, pp] + [vp] * 8
        lib.rglru_prefill_static_scratch.restype = i32
        lib.rglru_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
        lib.rglru_set_wait_limit_ns.restype = ctypes.c_uint64
        lib.rglru_query_status.argtypes = [vp, vp]
        lib.rglru_query_status.restype = i32
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().rglru_status_string(int(code)).decode()


def _io_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"io dtype must be float32 or bfloat16, got {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _chk(t: Optional[torch.Tensor], shape, dtype, name, device=None):
    if t is None:
        return
    if tuple(t.shape) != tuple(shape) or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name}: expected contiguous {dtype} tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)}")
    if device is not None and t.device != device:
        raise ValueError(f"{name}: expected device {device}, got {t.device}")


class Params:
    """Device-resident layer parameters: conv_w[4,D], conv_b[D]|None, W_a/W_x[H,Dh,Dh] (io dtype), b_a, b_x, lam [D] fp32."""

    def __init__(self, conv_w, conv_b, W_a, b_a, W_x, b_x, lam):
        H, Dh, Dh2 = W_a.shape
        D = H * Dh
        io = conv_w.dtype
        dev = conv_w.device
        _chk(conv_w, (4, D), io, "conv_w", dev); _chk(conv_b, (D,), torch.float32, "conv_b", dev)
        _chk(W_a, (H, Dh, Dh), io, "W_a", dev); _chk(W_x, (H, Dh, Dh), io, "W_x", dev)
        _chk(b_a, (D,), torch.float32, "b_a", dev); _chk(b_x, (D,), torch.float32, "b_x", dev)
        _chk(lam, (D,), torch.float32, "lam", dev)
        self.conv_w, self.conv_b, self.W_a, self.b_a, self.W_x, self.b_x, self.lam = conv_w, conv_b, W_a, b_a, W_x, b_x, lam
        self.H, self.D, self.io = H, D, io
        self.ptrs = ParamPtrs(conv_w.data_ptr(), 0 if conv_b is None else conv_b.data_ptr(), W_a.data_ptr(),
                              b_a.data_ptr(), W_x.data_ptr(), b_x.data_ptr(), lam.data_ptr())

    @classmethod
    def from_numpy(cls, p: dict, io: str, device="cuda"):
        """Upload a parameter dict of numpy arrays (values already representable in ``io``)."""
        dt = torch.bfloat16 if io == "bf16" else torch.float32
        up = lambda a, d: torch.from_numpy(a).to(device=device, dtype=d).contiguous()
        return cls(up(p["conv_w"], dt), None if p.get("conv_b") is None else up(p["conv_b"], torch.float32),
                   up(p["W_a"], dt), up(p["b_a"], torch.float32), up(p["W_x"], dt), up(p["b_x"], torch.float32),
                   up(p["lam"], torch.float32))


def make_shape(B, T, D, H, io_dtype: torch.dtype, c=8.0, flags=0) -> Shape:
    return Shape(B, T, D, H, BF16 if io_dtype == torch.bfloat16 else F32, float(c), int(flags))


def workspace_bytes(shape: Shape, op: int) -> int:
    return int(load().rglru_workspace_bytes(ctypes.byref(shape), op))


def alloc_workspace(shape: Shape, op: int, device) -> torch.Tensor:
    n = workspace_bytes(shape, op)
    if n == 0:
        raise RglruError(ERR_UNSUPPORTED, "rglru_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


class PrefillExtras(ctypes.Structure):
    _fields_ = [("gate_branch", ctypes.c_void_p), ("a_prod", ctypes.c_void_p)]


def prefill(x, params: Params, h0=None, conv_state_in=None, c=8.0, flags=0, y=None, h_T=None, conv_state_out=None,
            workspace=None, gate_branch=None, a_prod=None):
    """y, h_T, conv_state_out = Conv1D(4) + RG-LRU over x[B,T,D] (rglru_prefill; rglru_prefill_ex when an extra is given).
    ``gate_branch`` [B,T,D]: y_t = h_t * GeLU(gate_branch_t); ``a_prod`` [B,D] fp32 receives prod_t a_t."""
    lib = load()
    B, T, D = x.shape
    shape = make_shape(B, T, D, params.H, x.dtype, c, flags)
    dev = x.device
    _chk(x, (B, T, D), params.io, "x", params.conv_w.device)
    _chk(h0, (B, D), torch.float32, "h0", dev); _chk(conv_state_in, (B, 3, D), x.dtype, "conv_state_in", dev)
    y = torch.empty_like(x) if y is None else y
    h_T = torch.empty(B, D, dtype=torch.float32, device=dev) if h_T is None else h_T
    conv_state_out = torch.empty(B, 3, D, dtype=x.dtype, device=dev) if conv_state_out is None else conv_state_out
    _chk(y, (B, T, D), x.dtype, "y", dev); _chk(h_T, (B, D), torch.float32, "h_T", dev)
    _chk(conv_state_out, (B, 3, D), x.dtype, "conv_state_out", dev)
    _chk(gate_branch, (B, T, D), x.dtype, "gate_branch", dev); _chk(a_prod, (B, D), torch.float32, "a_prod", dev)
    ws = alloc_workspace(shape, OP_PREFILL, dev) if workspace is None else workspace
    if gate_branch is None and a_prod is None:
        rc = lib.rglru_prefill(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x), _ptr(h0), _ptr(conv_state_in),
                               _ptr(y), _ptr(h_T), _ptr(conv_state_out), _ptr(ws), ws.numel(), _stream())
    else:
        ex = PrefillExtras(_ptr(gate_branch), _ptr(a_prod))
        rc = lib.rglru_prefill_ex(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x), _ptr(h0), _ptr(conv_state_in),
                                  _ptr(y), _ptr(h_T), _ptr(conv_state_out), ctypes.byref(ex), _ptr(ws), ws.numel(), _stream())
    if rc != OK:
        raise RglruError(rc, "rglru_prefill")
    return y, h_T, conv_state_out


STATIC_SCRATCH_BYTES = 8 << 20


def prefill_static_scratch(x, params: Params, y, h_T, conv_state_out, h0=None, conv_state_in=None, c=8.0,
                           status_word=None):
    """rglru_prefill_static_scratch: the prefill for callers that cannot allocate device memory.  Every buffer,
    outputs included, comes from the caller; the kernel's scratch is an array inside the library (shared by all
    calls on the device, so calls must not overlap on the GPU).  ``status_word``: optional uint32 device tensor
    that receives a device-side timeout and can be passed to :func:`query_status`."""
    lib = load()
    B, T, D = x.shape
    shape = make_shape(B, T, D, params.H, x.dtype, c, 0)
    dev = x.device
    _chk(x, (B, T, D), params.io, "x", params.conv_w.device)
    _chk(h0, (B, D), torch.float32, "h0", dev); _chk(conv_state_in, (B, 3, D), x.dtype, "conv_state_in", dev)
    _chk(y, (B, T, D), x.dtype, "y", dev); _chk(h_T, (B, D), torch.float32, "h_T", dev)
    _chk(conv_state_out, (B, 3, D), x.dtype, "conv_state_out", dev)
    rc = lib.rglru_prefill_static_scratch(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x), _ptr(h0),
                                          _ptr(conv_state_in), _ptr(y), _ptr(h_T), _ptr(conv_state_out),
                                          _ptr(status_word), _stream())
    if rc != OK:
        raise RglruError(rc, "rglru_prefill_static_scratch")
    return y, h_T, conv_state_out


def decode_step(x, params: Params, h, conv_state, c=8.0, flags=0, y=None, workspace=None):
    """One token for B sequences; h[B,D] fp32 and conv_state[B,3,D] are updated in place; returns y[B,D]."""
    lib = load()
    B, D = x.shape
    shape = make_shape(B, 1, D, params.H, x.dtype, c, flags)
    dev = x.device
    _chk(x, (B, D), params.io, "x", params.conv_w.device); _chk(h, (B, D), torch.float32, "h", dev)
    _chk(conv_state, (B, 3, D), x.dtype, "conv_state", dev)
    y = torch.empty_like(x) if y is None else y
    _chk(y, (B, D), x.dtype, "y", dev)
    ws = alloc_workspace(shape, OP_DECODE, dev) if workspace is None else workspace
    rc = lib.rglru_decode_step(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x), _ptr(h), _ptr(conv_state),
                               _ptr(y), _ptr(ws), ws.numel(), _stream())
    if rc != OK:
        raise RglruError(rc, "rglru_decode_step")
    return y


class StateGrads(ctypes.Structure):
    _fields_ = [("dh_T", ctypes.c_void_p), ("dconv_state_out", ctypes.c_void_p), ("dh0", ctypes.c_void_p), ("dconv_state_in", ctypes.c_void_p)]


def backward(x, params: Params, dy, h0=None, conv_state_in=None, y=None, c=8.0, flags=0, workspace=None, out=None,
             dh_T=None, dconv_state_out=None, state_grads=False):
    """Gradients of sum(dy*y) [+ sum(dh_T*h_T) + sum(dconv_state_out*conv_state_out)] (rglru_backward): dict with x (io dtype)
    and fp32 conv_w, conv_b, W_a, b_a, W_x, b_x, lam; with ``state_grads`` also h0 [B,D] fp32 and conv_state [B,3,D] io."""
    lib = load()
    B, T, D = x.shape
    H, Dh = params.H, D // params.H
    shape = make_shape(B, T, D, H, x.dtype, c, flags)
    dev = x.device
    _chk(x, (B, T, D), params.io, "x", params.conv_w.device); _chk(dy, (B, T, D), x.dtype, "dy", dev)
    _chk(y, (B, T, D), x.dtype, "y", dev)
    _chk(h0, (B, D), torch.float32, "h0", dev); _chk(conv_state_in, (B, 3, D), x.dtype, "conv_state_in", dev)
    f32 = dict(dtype=torch.float32, device=dev)
    g = dict(x=torch.empty_like(x), conv_w=torch.empty(4, D, **f32), conv_b=torch.empty(D, **f32),
             W_a=torch.empty(H, Dh, Dh, **f32), b_a=torch.empty(D, **f32), W_x=torch.empty(H, Dh, Dh, **f32),
             b_x=torch.empty(D, **f32), lam=torch.empty(D, **f32))
    if out is not None:   # caller-provided gradient buffers (same keys, shapes and dtypes)
        for k in g:
            _chk(out[k], tuple(g[k].shape), g[k].dtype, "out[" + k + "]", dev)
        g = out
    ws = alloc_workspace(shape, OP_BACKWARD, dev) if workspace is None else workspace
    _chk(dh_T, (B, D), torch.float32, "dh_T", dev); _chk(dconv_state_out, (B, 3, D), x.dtype, "dconv_state_out", dev)
    sg = None
    if state_grads or dh_T is not None or dconv_state_out is not None:
        if state_grads and (out is None or "h0" not in out):
            g["h0"] = torch.empty(B, D, **f32); g["conv_state"] = torch.empty(B, 3, D, dtype=x.dtype, device=dev)
        vp = lambda t: None if t is None else t.data_ptr()
        sg = StateGrads(vp(dh_T), vp(dconv_state_out), vp(g.get("h0")), vp(g.get("conv_state")))
    rc = lib.rglru_backward(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x), _ptr(h0), _ptr(conv_state_in),
                            _ptr(y), _ptr(dy), _ptr(g["x"]), _ptr(g["conv_w"]), _ptr(g["conv_b"]), _ptr(g["W_a"]),
                            _ptr(g["b_a"]), _ptr(g["W_x"]), _ptr(g["b_x"]), _ptr(g["lam"]),
                            ctypes.byref(sg) if sg is not None else None, _ptr(ws), ws.numel(), _stream())
    if rc != OK:
        raise RglruError(rc, "rglru_backward")
    return g


def host_staging_bytes(shape: Shape) -> int:
    return int(load().rglru_host_staging_bytes(ctypes.byref(shape)))


def prefill_host(x_host, params: Params, y_host, h_T_host, conv_state_out_host, staging, workspace, h0=None,
                 conv_state_in=None, c=8.0, flags=0):
    """rglru_prefill_host: activations in (pinned) host tensors, copies and kernels enqueued on the current stream."""
    lib = load()
    B, T, D = x_host.shape
    shape = make_shape(B, T, D, params.H, x_host.dtype, c, flags)
    for t, n in ((x_host, "x_host"), (y_host, "y_host"), (h_T_host, "h_T_host"), (conv_state_out_host, "conv_state_out_host")):
        if t.device.type != "cpu" or not t.is_contiguous():
            raise ValueError(f"{n} must be a contiguous host tensor")
    rc = lib.rglru_prefill_host(ctypes.byref(shape), ctypes.byref(params.ptrs), _ptr(x_host), _ptr(h0), _ptr(conv_state_in),
                                _ptr(y_host), _ptr(h_T_host), _ptr(conv_state_out_host), _ptr(staging), staging.numel(),
                                _ptr(workspace), workspace.numel(), _stream())
    if rc != OK:
        raise RglruError(rc, "rglru_prefill_host")


def set_wait_limit_ns(ns: int) -> int:
    """Time limit of device-side waits (0 restores the 2 s default); returns the previous value."""
    return int(load().rglru_set_wait_limit_ns(int(ns)))


def query_status(workspace) -> int:
    return int(load().rglru_query_status(_ptr(workspace), _stream()))
