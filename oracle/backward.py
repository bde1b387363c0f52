"""CPU oracle for the BACKWARD pass of the Slide Attention forward -- TEST INFRASTRUCTURE ONLY.

The paper trains every model through the module (Sec. 4.3, Fig. 4 (1); training setup in App. B) but
prints no backward formulas: the gradients are the derivatives of Eq. 2 with the depthwise
convolution of Eq. 12 inside, written out here by the chain rule, step by step in the forward's own
order run backwards, in double precision with plain array arithmetic (one statement per formula,
loops over slots and taps):

  forward   Ks[s] = sum_t wk[:, s, t] * shift_t(k)            Eq. 12 (zero padding, no kernel flip)
            l[s]  = (q . Ks[s]) / sqrt(d) + bias[h, s]         Eq. 2
            a     = softmax_s(l);  out = sum_s a[s] Vs[s]      Eq. 2
  backward  dVs[s] = a[s] g                da[s] = g . Vs[s]
            dl[s]  = a[s] (da[s] - sum_s' a[s'] da[s'])         (softmax)
            dbias[h, s] = sum over pixels of dl[s]
            dq     = sum_s dl[s] Ks[s] / sqrt(d)       dKs[s] = dl[s] q / sqrt(d)
            dwk[c, s, t] = sum over pixels of dKs[s][c] * shift_t(k)[c]
            dk     = sum_{s,t} shift_t^T( wk[:, s, t] * dKs[s] )      (the transpose of the shift:
                     what a pixel received from offset t goes back to the pixel at that offset;
                     what came from the padding is dropped)
            and the same two lines for wv / v with dVs.

`merged = shift + learned` (Sec. 4.3), so the gradient of the learned kernels of the training-time
two-path form equals the gradient of the merged kernels; `two_path_backward` states that.

Pinned by tests/test_oracle_backward.py: central finite differences of `oracle.forward` on inputs
chosen so that x +- eps is exact in float, the two-path identity, k = 1, and the softmax invariants.
Nothing here is used by the library.
"""
from __future__ import annotations

import numpy as np


def _shifted(f, ksize):
    """shift_t(f) for every tap t: [k*k][B,H,W,C], zero where the tap leaves the map (Fig. 2)."""
    B, H, W, C = f.shape
    r = ksize // 2
    fp = np.zeros((B, H + 2 * r, W + 2 * r, C))
    fp[:, r:r + H, r:r + W] = f
    return [fp[:, p:p + H, q_:q_ + W, :] for p in range(ksize) for q_ in range(ksize)]


def _unshift_add(dst, g, t, ksize):
    """dst[pixel + off(t)] += g[pixel] for every pixel whose tap t lies inside the map."""
    B, H, W, C = g.shape
    r = ksize // 2
    dp = np.zeros((B, H + 2 * r, W + 2 * r, C))
    p, q_ = divmod(t, ksize)
    dp[:, p:p + H, q_:q_ + W, :] = g
    dst += dp[:, r:r + H, r:r + W, :]


def backward(q, k, v, wk, wv, bias, ksize, dout):
    """Gradients of sum(out * dout) w.r.t. every input of the forward.  Shapes as the forward's;
    returns dict(dq, dk, dv, dwk, dwv, dbias) in double (dbias None without bias)."""
    q, k, v, wk, wv, g = (np.asarray(a, dtype=np.float64) for a in (q, k, v, wk, wv, dout))
    B, H, W, heads, d = q.shape
    C, k2 = heads * d, ksize * ksize
    kc, vc, gc, qc = (a.reshape(B, H, W, C) for a in (k, v, g, q))
    ksh, vsh = _shifted(kc, ksize), _shifted(vc, ksize)
    # forward, kept: Ks, Vs [k2][B,H,W,C]; a [B,H,W,heads,k2]
    Ks = [sum(wk[:, s, t] * ksh[t] for t in range(k2)) for s in range(k2)]
    Vs = [sum(wv[:, s, t] * vsh[t] for t in range(k2)) for s in range(k2)]
    l = np.stack([(qc * Ks[s]).reshape(B, H, W, heads, d).sum(-1) for s in range(k2)], -1) / np.sqrt(float(d))
    if bias is not None:
        l = l + np.asarray(bias, dtype=np.float64)
    e = np.exp(l - l.max(-1, keepdims=True))
    a = e / e.sum(-1, keepdims=True)
    # backward
    da = np.stack([(gc * Vs[s]).reshape(B, H, W, heads, d).sum(-1) for s in range(k2)], -1)
    dl = a * (da - (a * da).sum(-1, keepdims=True))
    dbias = None if bias is None else dl.sum((0, 1, 2))
    per_channel = lambda x: np.repeat(x, d, axis=-1)            # [B,H,W,heads] -> [B,H,W,C]
    dq = sum(per_channel(dl[..., s]) * Ks[s] for s in range(k2)) / np.sqrt(float(d))
    dKs = [per_channel(dl[..., s]) * qc / np.sqrt(float(d)) for s in range(k2)]
    dVs = [per_channel(a[..., s]) * gc for s in range(k2)]
    dwk, dwv = np.zeros_like(wk), np.zeros_like(wv)
    dk, dv = np.zeros_like(kc), np.zeros_like(vc)
    for s in range(k2):
        for t in range(k2):
            dwk[:, s, t] = (dKs[s] * ksh[t]).sum((0, 1, 2))
            dwv[:, s, t] = (dVs[s] * vsh[t]).sum((0, 1, 2))
            _unshift_add(dk, wk[:, s, t] * dKs[s], t, ksize)
            _unshift_add(dv, wv[:, s, t] * dVs[s], t, ksize)
    return dict(dq=dq.reshape(q.shape), dk=dk.reshape(q.shape), dv=dv.reshape(q.shape), dwk=dwk, dwv=dwv, dbias=dbias)


def two_path_backward(q, k, v, shift_w, learned_wk, learned_wv, bias, ksize, dout):
    """Training-time form (Fig. 4 (1)): the fixed-shift kernels are constants, the learned kernels the
    parameters.  The two paths add before the attention, so the learned kernels' gradient is the merged
    kernels' gradient; everything else is the merged form's."""
    g = backward(q, k, v, np.asarray(shift_w, np.float64) + np.asarray(learned_wk, np.float64),
                 np.asarray(shift_w, np.float64) + np.asarray(learned_wv, np.float64), bias, ksize, dout)
    g["dlearned_wk"], g["dlearned_wv"] = g.pop("dwk"), g.pop("dwv")
    return g
