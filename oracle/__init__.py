"""ctypes front end of the fp64 CPU oracle (``rglru_oracle.c``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library and its Python binding never do, and this
package imports nothing of theirs.  All arrays are float64 numpy arrays; callers convert
stored fp32 / bf16 values exactly before calling.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rglru_oracle.c")
_LIB = os.path.join(_HERE, "librglru_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_dp = ctypes.POINTER(ctypes.c_double)


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_decay.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double, _dp, _dp]
        lib.oracle_decay.restype = None
        lib.oracle_prefill.argtypes = [ctypes.c_int] * 4 + [ctypes.c_double] + [_dp] * 15
        lib.oracle_prefill.restype = ctypes.c_int
        lib.oracle_gelu.argtypes = [ctypes.c_double]
        lib.oracle_gelu.restype = ctypes.c_double
        lib.oracle_decode_step.argtypes = [ctypes.c_int] * 3 + [ctypes.c_double] + [_dp] * 11
        lib.oracle_decode_step.restype = ctypes.c_int
        lib.oracle_backward.argtypes = [ctypes.c_int] * 4 + [ctypes.c_double] + [_dp] * 23
        lib.oracle_backward.restype = ctypes.c_int
        _lib = lib
    return _lib


def _in(a, shape):
    """float64, C-contiguous, checked shape; None passes through as NULL."""
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a, a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def decay(lam: float, r: float, c: float = 8.0):
    """(a_t, sqrt(1-a_t^2)) for one channel: Eq. 3 in log space (Appendix A)."""
    a = ctypes.c_double()
    m = ctypes.c_double()
    _load().oracle_decay(float(lam), float(r), float(c), ctypes.byref(a), ctypes.byref(m))
    return a.value, m.value


def _params(p, D, H):
    Dh = D // H
    keep, ptrs = [], []
    for name, shape in (("conv_w", (4, D)), ("conv_b", (D,)), ("W_a", (H, Dh, Dh)), ("b_a", (D,)),
                        ("W_x", (H, Dh, Dh)), ("b_x", (D,)), ("lam", (D,))):
        arr, ptr = _in(p.get(name), shape)
        if arr is None and name != "conv_b":
            raise ValueError(f"missing parameter {name}")
        keep.append(arr)
        ptrs.append(ptr)
    return keep, ptrs


def gelu(v: float) -> float:
    """GeLU(v) = v Phi(v) (Section 2.3: the non-linearity on the recurrent block's second branch)."""
    return float(_load().oracle_gelu(float(v)))


def prefill(x, params, H, c=8.0, h0=None, conv_state_in=None, gate_branch=None, with_a_prod=False):
    """Conv1D(4) + RG-LRU over T tokens (Eq. 1-4).  Returns (y[B,T,D], h_T[B,D], conv_state_out[B,3,D]), and with
    ``with_a_prod`` a fourth array prod_t a_t [B,D].  With ``gate_branch`` [B,T,D], y_t = h_t * GeLU(gate_branch_t)
    (Section 2.3) while h_T stays the raw state."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, T, D = x.shape
    keep, (cw, cb, Wa, ba, Wx, bx, lam) = _params(params, D, H)
    h0a, h0p = _in(h0, (B, D))
    csa, csp = _in(conv_state_in, (B, 3, D))
    gba, gbp = _in(gate_branch, (B, T, D))
    y = np.empty((B, T, D)); hT = np.empty((B, D)); cso = np.empty((B, 3, D))
    ap = np.empty((B, D)) if with_a_prod else None
    rc = _load().oracle_prefill(B, T, D, H, float(c), x.ctypes.data_as(_dp), cw, cb, Wa, ba, Wx, bx, lam, h0p, csp,
                                y.ctypes.data_as(_dp), hT.ctypes.data_as(_dp), cso.ctypes.data_as(_dp), gbp,
                                ap.ctypes.data_as(_dp) if with_a_prod else None)
    if rc != 0:
        raise ValueError("oracle_prefill: bad shape")
    return (y, hT, cso, ap) if with_a_prod else (y, hT, cso)


def decode_step(x, params, H, h, conv_state, c=8.0):
    """One token for B sequences; returns (y[B,D], h_new[B,D], conv_state_new[B,3,D]) (inputs are not modified)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, D = x.shape
    keep, (cw, cb, Wa, ba, Wx, bx, lam) = _params(params, D, H)
    h = np.array(h, dtype=np.float64, order="C", copy=True)
    cs = np.array(conv_state, dtype=np.float64, order="C", copy=True)
    if h.shape != (B, D) or cs.shape != (B, 3, D):
        raise ValueError("bad state shape")
    y = np.empty((B, D))
    rc = _load().oracle_decode_step(B, D, H, float(c), x.ctypes.data_as(_dp), cw, cb, Wa, ba, Wx, bx, lam,
                                    h.ctypes.data_as(_dp), cs.ctypes.data_as(_dp), y.ctypes.data_as(_dp))
    if rc != 0:
        raise ValueError("oracle_decode_step: bad shape")
    return y, h, cs


def backward(x, params, H, dy, c=8.0, h0=None, conv_state_in=None, dh_T=None, dconv_state_out=None, state_grads=False):
    """Gradients of sum(dy*y) [+ sum(dh_T*h_T) + sum(dconv_state_out*conv_state_out)] w.r.t. x and every parameter; returns
    a dict keyed like ``params`` plus 'x', and with ``state_grads`` also 'h0' [B,D] and 'conv_state' [B,3,D]."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, T, D = x.shape
    Dh = D // H
    keep, (cw, cb, Wa, ba, Wx, bx, lam) = _params(params, D, H)
    h0a, h0p = _in(h0, (B, D))
    csa, csp = _in(conv_state_in, (B, 3, D))
    dya, dyp = _in(dy, (B, T, D))
    out = {"x": np.empty((B, T, D)), "conv_w": np.empty((4, D)), "conv_b": np.empty((D,)),
           "W_a": np.empty((H, Dh, Dh)), "b_a": np.empty((D,)), "W_x": np.empty((H, Dh, Dh)),
           "b_x": np.empty((D,)), "lam": np.empty((D,))}
    if state_grads:
        out["h0"] = np.empty((B, D)); out["conv_state"] = np.empty((B, 3, D))
    P = {k: v.ctypes.data_as(_dp) for k, v in out.items()}
    dha, dhp = _in(dh_T, (B, D))
    dca, dcp = _in(dconv_state_out, (B, 3, D))
    rc = _load().oracle_backward(B, T, D, H, float(c), x.ctypes.data_as(_dp), cw, cb, Wa, ba, Wx, bx, lam, h0p, csp, dyp,
                                 P["x"], P["conv_w"], P["conv_b"], P["W_a"], P["b_a"], P["W_x"], P["b_x"], P["lam"],
                                 dhp, dcp, P.get("h0"), P.get("conv_state"))
    if rc != 0:
        raise ValueError("oracle_backward: bad shape")
    return out
