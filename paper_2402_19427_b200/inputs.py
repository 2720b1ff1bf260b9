"""Seeded synthetic inputs for the RG-LRU temporal core.

This module serves both the CUDA path and the CPU oracle and therefore holds none of the
method's arithmetic: it only draws random tensors, applies the paper's initialisation
rules (Section 2.4: LeCun-normal gate weights, Lambda such that a^c = sigmoid(Lambda)^c is
uniform in [0.9, 0.999]) and rounds values to the storage dtype.  numpy only.

Values are returned as float32 numpy arrays that are exactly representable in the storage
dtype ("f32" or "bf16"), so the oracle (after an exact widening to float64) and the GPU
(after an exact narrowing to bf16 bits) see the same numbers.
"""
from __future__ import annotations

import numpy as np

# The five benchmark / parity workloads.  Shapes follow the paper's model table
# (Appendix C: RNN widths 2560 and 4096 are the 1.3B and 3B models), its training
# sequence length (2048) and its long-context evaluations.
CONFIGS = {
    0: dict(name="tiny_fp32", B=1, T=256, D=256, H=2, io="f32"),
    1: dict(name="train_prefill", B=8, T=2048, D=2560, H=10, io="bf16"),
    2: dict(name="long_prefill", B=1, T=65536, D=4096, H=16, io="bf16", long_memory_frac=0.05),
    3: dict(name="batched_decode", B=512, T=768, D=2560, H=10, io="bf16", prefill_T=512, decode_steps=256),
    4: dict(name="train_fwd_bwd", B=4, T=4096, D=4096, H=16, io="bf16", with_dy=True),
}
BASE_SEED = 20240219


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already exactly representable in bf16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    if np.any(bits & np.uint32(0xFFFF)):
        raise ValueError("value not representable in bf16")
    return (bits >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """float32 values of uint16 bf16 bit patterns."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(a: np.ndarray, io: str) -> np.ndarray:
    a = np.asarray(a, dtype=np.float32)
    return round_to_bf16(a) if io == "bf16" else np.ascontiguousarray(a)


def lambda_for_decay(a_pow_c: np.ndarray, c: float = 8.0) -> np.ndarray:
    """Lambda with sigmoid(Lambda)^c == a_pow_c, i.e. Lambda = logit(a_pow_c^(1/c)) (Section 2.4 init rule)."""
    a = np.asarray(a_pow_c, dtype=np.float64) ** (1.0 / c)
    return np.log(a) - np.log1p(-a)


def make_inputs(B, T, D, H, io="bf16", seed=BASE_SEED, long_memory_frac=0.0, with_dy=False,
                with_state=False, bias_scale=0.0, c=8.0):
    """Draw one workload.  Draw order is fixed: x, conv_w, W_a, W_x, u_Lambda, [long-memory mask], [dy], [state], [biases].

    Returns a dict: x[B,T,D], params{conv_w[4,D], conv_b[D], W_a[H,Dh,Dh], b_a[D], W_x[H,Dh,Dh], b_x[D], lam[D]},
    optionally dy[B,T,D], h0[B,D], conv_state[B,3,D]; plus shape fields.  Matrices are rounded to ``io``;
    per-channel vectors (biases, Lambda, h0) stay fp32.
    """
    if D % H:
        raise ValueError("D must be a multiple of H")
    Dh = D // H
    rng = np.random.Generator(np.random.PCG64(seed))
    x = _store(rng.standard_normal((B, T, D), dtype=np.float32), io)
    conv_w = _store(rng.standard_normal((4, D), dtype=np.float32) * 0.5, io)          # N(0, 1/4): Var(u) ~ 1
    W_a = _store(rng.standard_normal((H, Dh, Dh), dtype=np.float32) / np.sqrt(Dh), io)  # LeCun normal, fan-in Dh
    W_x = _store(rng.standard_normal((H, Dh, Dh), dtype=np.float32) / np.sqrt(Dh), io)
    a_pow_c = rng.uniform(0.9, 0.999, size=D)
    if long_memory_frac > 0.0:
        n_long = int(round(long_memory_frac * D))
        idx = rng.permutation(D)[:n_long]
        a_pow_c[idx] = 0.9999
    lam = lambda_for_decay(a_pow_c, c).astype(np.float32)
    out = dict(B=B, T=T, D=D, H=H, io=io, c=float(c), seed=seed, x=x)
    if with_dy:
        out["dy"] = _store(rng.standard_normal((B, T, D), dtype=np.float32), io)
    if with_state:
        out["h0"] = rng.standard_normal((B, D), dtype=np.float32)
        out["conv_state"] = _store(rng.standard_normal((B, 3, D), dtype=np.float32), io)
    if bias_scale > 0.0:
        conv_b = (rng.standard_normal(D, dtype=np.float32) * bias_scale).astype(np.float32)
        b_a = (rng.standard_normal(D, dtype=np.float32) * bias_scale).astype(np.float32)
        b_x = (rng.standard_normal(D, dtype=np.float32) * bias_scale).astype(np.float32)
    else:
        conv_b = np.zeros(D, np.float32); b_a = np.zeros(D, np.float32); b_x = np.zeros(D, np.float32)
    out["params"] = dict(conv_w=conv_w, conv_b=conv_b, W_a=W_a, b_a=b_a, W_x=W_x, b_x=b_x, lam=lam)
    return out


def make_config(cfg_id: int, **overrides):
    """Inputs of one of the five named workloads (seed = BASE_SEED + cfg_id unless overridden)."""
    cfg = dict(CONFIGS[cfg_id])
    cfg.pop("name")
    cfg.pop("prefill_T", None)
    cfg.pop("decode_steps", None)
    cfg.setdefault("seed", BASE_SEED + cfg_id)
    cfg.update(overrides)
    return make_inputs(**cfg)


def head_slice(inp: dict, heads, batches=None) -> dict:
    """Restrict a workload to some heads (and batch rows).  Heads are independent (block-diagonal gates,
    depthwise conv, diagonal recurrence), so a slice is a self-contained smaller workload."""
    heads = list(heads)
    D, H = inp["D"], inp["H"]
    Dh = D // H
    ch = np.concatenate([np.arange(k * Dh, (k + 1) * Dh) for k in heads])
    bsel = slice(None) if batches is None else list(batches)
    p = inp["params"]
    out = dict(inp)
    out["x"] = np.ascontiguousarray(inp["x"][bsel][:, :, ch])
    out["B"] = out["x"].shape[0]
    out["D"] = len(ch)
    out["H"] = len(heads)
    for k in ("dy",):
        if k in inp:
            out[k] = np.ascontiguousarray(inp[k][bsel][:, :, ch])
    if "h0" in inp:
        out["h0"] = np.ascontiguousarray(inp["h0"][bsel][:, ch])
    if "conv_state" in inp:
        out["conv_state"] = np.ascontiguousarray(inp["conv_state"][bsel][:, :, ch])
    out["params"] = dict(conv_w=np.ascontiguousarray(p["conv_w"][:, ch]), conv_b=p["conv_b"][ch].copy(),
                         W_a=np.ascontiguousarray(p["W_a"][heads]), b_a=p["b_a"][ch].copy(),
                         W_x=np.ascontiguousarray(p["W_x"][heads]), b_x=p["b_x"][ch].copy(), lam=p["lam"][ch].copy())
    return out
