"""CPU oracle of a whole Slide-Attention block -- TEST INFRASTRUCTURE ONLY.

The block is multi-head self-attention (Eq. 1-3) with the local attention of this paper as its middle
stage: the projections q = x W_q, k = x W_k, v = x W_v (Eq. 1), per head the attention over the k x k
window with keys and values from the merged depthwise convolution (Eq. 2 with Sec. 4.2 / 4.3 inside:
`oracle.forward`), and the output projection Concat(heads) W_o (Eq. 3).  Channel c of a projected
tensor belongs to head c // d, element c % d.

Everything is evaluated in double precision with numpy's matrix product as the only library step.
`storage="bf16"` states where a block that keeps its intermediate tensors in bf16 rounds: q, k, v once
after Eq. 1 and the attention output once before Eq. 3, each to the nearest bf16 (ties to even); the
paper is silent on intermediate precision, "f64" rounds nowhere.

Pinned by tests/test_oracle_block.py (brute-force loops over Eq. 1 and Eq. 3, identity projections
against `oracle.forward`, the 1 x 1 closed form, a channel permutation that moves heads, the rounding
helper against a library conversion); nothing here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

import oracle


def round_bf16(a):
    """Nearest bf16 (ties to even) of every element, returned as float64."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    keep = (u >> np.uint32(16)) & np.uint32(1)
    u = (u + np.uint32(0x7FFF) + keep) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def project(x, w):
    """Eq. 1 / Eq. 3 for one weight: x [..., C_in], w [C_in, C_out] -> [..., C_out] in double."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    assert x.shape[-1] == w.shape[0]
    return x @ w


def block_forward(x, w_q, w_k, w_v, w_o, wk, wv, bias, ksize, heads, storage="f64", return_parts=False):
    """x [B,H,W,C]; w_q, w_k, w_v, w_o [C,C] (input channel, output channel); wk, wv [C,k*k,k*k];
    bias [heads,k*k] or None.  Returns the block output [B,H,W,C] in double (and q, k, v, z)."""
    assert storage in ("f64", "bf16")
    x = np.asarray(x, dtype=np.float64)
    B, H, W, C = x.shape
    assert C % heads == 0
    d = C // heads
    rnd = round_bf16 if storage == "bf16" else (lambda a: a)
    # Eq. 1
    q = rnd(project(x, w_q)).reshape(B, H, W, heads, d)
    k = rnd(project(x, w_k)).reshape(B, H, W, heads, d)
    v = rnd(project(x, w_v)).reshape(B, H, W, heads, d)
    # Eq. 2 per head, local window, deformed shift inside.  The C oracle takes float inputs: exact for
    # bf16-rounded values; for "f64" the projections are narrowed to float first.
    z = oracle.forward(q.astype(np.float32), k.astype(np.float32), v.astype(np.float32), wk, wv, bias, ksize)
    z = rnd(z).reshape(B, H, W, C)
    # Eq. 3
    out = project(z, w_o)
    return (out, q, k, v, z) if return_parts else out
