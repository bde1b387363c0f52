"""Seeded synthetic inputs for the Slide Attention forward.

This module holds data generation only: a counter-based random stream, rounding
of host values to the storage dtype, and the table of workload shapes.  None of
the method's arithmetic (convolution, logits, softmax, aggregation) lives here,
so both the CUDA path's tests and the CPU oracle's tests may draw from it.

Workload shapes stand in for feature maps of hierarchical vision transformers
(the architecture tables of the paper's appendix): 56x56 maps with 64 or 96
channels (stage 1), 28x28 with 192 channels (stage 2), and a 128x128 map as a
dense-prediction crop at stride 4.  Values: q, k, v are i.i.d. N(0,1), rounded
to the storage dtype; the merged depthwise weights are the one-hot shift kernel
of each slot (Eq. 11) plus sigma_w * N(0,1) (the learned deformed-shift path,
Sec. 4.3, after re-parameterisation); the optional per-slot bias is
sigma_b * N(0,1).
"""
from __future__ import annotations

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix64(z: np.ndarray) -> np.ndarray:
    """The splitmix64 output function on an array of uint64 counters."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def uniform01(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in (0,1): element i depends only on (seed, stream, offset+i)."""
    with np.errstate(over="ignore"):
        base = _mix64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + _GAMMA * np.uint64(stream + 1))
        idx = np.arange(offset, offset + n, dtype=np.uint64)
        bits = _mix64(base + _GAMMA * (idx + np.uint64(1)))
    # 53 random mantissa bits, shifted half a step away from 0
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """n standard normals (float64) by Box-Muller over two counter streams."""
    chunk = 1 << 22
    out = np.empty(n, dtype=np.float64)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        u1 = uniform01(seed, 2 * stream, m, lo)
        u2 = uniform01(seed, 2 * stream + 1, m, lo)
        out[lo:lo + m] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array -> float32 array holding the nearest-even bf16 values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 array of bf16-representable values -> uint16 bit patterns."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# name -> shape and recipe.  "c3_k5" etc. are the neighbourhood-size sweeps.
def _cfg(B, H, W, heads, d, k, dtype, sigma_w, bias, cid, variant=0):
    return dict(B=B, H=H, W=W, heads=heads, head_dim=d, ksize=k, dtype=dtype,
                sigma_w=sigma_w, sigma_b=0.02, has_bias=bias,
                seed=0x51DE0000 + 16 * cid + variant)


CONFIGS = {
    "c1_tiny":   _cfg(1, 14, 14, 1, 32, 3, "f32", 0.02, False, 1),
    "c2":        _cfg(64, 56, 56, 2, 32, 3, "bf16", 0.02, True, 2),
    "c3":        _cfg(64, 56, 56, 3, 32, 3, "bf16", 0.02, True, 3),
    "c3_k5":     _cfg(64, 56, 56, 3, 32, 5, "bf16", 0.02, True, 3, 1),
    "c3_k7":     _cfg(64, 56, 56, 3, 32, 7, "bf16", 0.02, True, 3, 2),
    "c4":        _cfg(64, 28, 28, 6, 32, 3, "bf16", 0.02, True, 4),
    "c4_ragged": _cfg(32, 28, 42, 6, 32, 3, "bf16", 0.02, True, 4, 1),
    "c5":        _cfg(2, 128, 128, 3, 32, 3, "bf16", 0.05, True, 5),
    "c5_k5":     _cfg(2, 128, 128, 3, 32, 5, "bf16", 0.05, True, 5, 1),
    "c5_k7":     _cfg(2, 128, 128, 3, 32, 7, "bf16", 0.05, True, 5, 2),
    "c5_k9":     _cfg(2, 128, 128, 3, 32, 9, "bf16", 0.05, True, 5, 3),
    "c5_f32":    _cfg(2, 128, 128, 3, 32, 3, "f32", 0.05, False, 5, 4),
}


def one_hot_weights(C: int, ksize: int) -> np.ndarray:
    """The fixed shift kernels: w[c, slot, tap] = 1 where tap == slot (Eq. 11)."""
    k2 = ksize * ksize
    w = np.zeros((C, k2, k2), dtype=np.float32)
    idx = np.arange(k2)
    w[:, idx, idx] = 1.0
    return w


def make_inputs(B, H, W, heads, head_dim, ksize, dtype="f32", sigma_w=0.02, sigma_b=0.02,
                has_bias=False, seed=0, batch_limit=None, **_):
    """Host inputs as float32 arrays holding exactly the stored values.

    Returns dict(q, k, v [B,H,W,heads,head_dim]; wk, wv [C,k*k,k*k]; bias
    [heads,k*k] or None).  Draw order: q, k, v, wk, wv, bias; element order is
    memory order, so `batch_limit` images are a prefix of the full tensors.
    """
    C = heads * head_dim
    k2 = ksize * ksize
    Bn = B if batch_limit is None else min(B, batch_limit)
    n = Bn * H * W * C
    shape = (Bn, H, W, heads, head_dim)
    out = {}
    for stream, name in enumerate(("q", "k", "v")):
        x = normal(seed, stream, n).astype(np.float32)
        if dtype == "bf16":
            x = round_to_bf16(x)
        out[name] = x.reshape(shape)
    for stream, name in ((3, "wk"), (4, "wv")):
        dlt = (sigma_w * normal(seed, stream, C * k2 * k2)).astype(np.float32).reshape(C, k2, k2)
        out[name] = one_hot_weights(C, ksize) + dlt
    out["bias"] = ((sigma_b * normal(seed, 5, heads * k2)).astype(np.float32).reshape(heads, k2)
                   if has_bias else None)
    return out


def make_config(name: str, batch_limit=None):
    cfg = CONFIGS[name]
    return cfg, make_inputs(batch_limit=batch_limit, **cfg)
