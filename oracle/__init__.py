"""CPU oracle for the Slide Attention forward -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  The library (the CUDA path and its Python binding) never does,
and nothing here imports the library.

Contents
  * `forward`, `forward_pixels`, `dwconv`: ctypes wrappers of the plain-C,
    double-precision definition in `slide_attn_oracle.c` (Eq. 2 with the k x k
    window as receptive field; keys and values per slot from the merged
    depthwise convolution of Sec. 4.2 / 4.3).
  * `im2col_local_attention`: the column-view definition (Eq. 4-7): explicit
    gather of every query's k x k window, then dense attention on it.  Valid for
    the fixed-shift kernels only.  Pure Python loops; tiny inputs only.
  * `two_path_forward`: the training-time form of the deformed shifting module
    (Fig. 4 (1)): fixed-shift path and learned path evaluated separately and
    summed, then the same attention.

All of these are pinned by tests/test_oracle_pins.py against closed forms,
brute force and library routines; none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slide_attn_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libslide_attn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", _SRC,
                        "-o", tmp, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        fp, dp, ip = (ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double),
                      ctypes.POINTER(ctypes.c_longlong))
        i = ctypes.c_int
        lib.slide_attn_oracle.argtypes = [fp] * 6 + [i] * 6 + [dp, dp]
        lib.slide_attn_oracle.restype = i
        lib.slide_attn_oracle_pixels.argtypes = [fp] * 6 + [i] * 6 + [ip, ctypes.c_longlong, dp]
        lib.slide_attn_oracle_pixels.restype = i
        lib.slide_attn_oracle_dwconv.argtypes = [fp, fp] + [i] * 5 + [dp]
        lib.slide_attn_oracle_dwconv.restype = i
        lib.slide_attn_oracle_threads.restype = i
        _lib = lib
    return _lib


def threads() -> int:
    """Host threads the C oracle uses (OpenMP default)."""
    return int(_load().slide_attn_oracle_threads())


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a, ty):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ty))


def _prep(q, k, v, wk, wv, bias, ksize):
    q, k, v, wk, wv, bias = map(_f32, (q, k, v, wk, wv, bias))
    B, H, W, heads, d = q.shape
    k2 = ksize * ksize
    assert k.shape == q.shape and v.shape == q.shape
    assert wk.shape == (heads * d, k2, k2) and wv.shape == wk.shape
    assert bias is None or bias.shape == (heads, k2)
    return (q, k, v, wk, wv, bias), (B, H, W, heads, d, ksize)


def forward(q, k, v, wk, wv, bias=None, ksize=3, return_attn=False):
    """Full forward in double.  q,k,v [B,H,W,heads,d]; returns out (and attn)."""
    arrs, dims = _prep(q, k, v, wk, wv, bias, ksize)
    B, H, W, heads, d, _ = dims
    out = np.empty((B, H, W, heads, d), dtype=np.float64)
    attn = np.empty((B, H, W, heads, ksize * ksize), dtype=np.float64) if return_attn else None
    rc = _load().slide_attn_oracle(*[_ptr(a, ctypes.c_float) for a in arrs], *dims,
                                   _ptr(out, ctypes.c_double), _ptr(attn, ctypes.c_double))
    if rc != 0:
        raise ValueError("slide_attn_oracle: invalid arguments")
    return (out, attn) if return_attn else out


def forward_pixels(q, k, v, wk, wv, bias, ksize, pix):
    """The definition at the flat pixel indices `pix`; returns [len(pix), heads*d]."""
    arrs, dims = _prep(q, k, v, wk, wv, bias, ksize)
    pix = np.ascontiguousarray(pix, dtype=np.int64)
    out = np.empty((pix.size, dims[3] * dims[4]), dtype=np.float64)
    rc = _load().slide_attn_oracle_pixels(*[_ptr(a, ctypes.c_float) for a in arrs], *dims,
                                          _ptr(pix, ctypes.c_longlong), pix.size,
                                          _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("slide_attn_oracle_pixels: invalid arguments")
    return out


def dwconv(f, w, ksize):
    """Step 1 alone (Eq. 12, all slots): f [B,H,W,C], w [C,k*k,k*k] -> [B,H,W,k*k,C]."""
    f, w = _f32(f), _f32(w)
    B, H, W, C = f.shape
    out = np.empty((B, H, W, ksize * ksize, C), dtype=np.float64)
    rc = _load().slide_attn_oracle_dwconv(_ptr(f, ctypes.c_float), _ptr(w, ctypes.c_float),
                                          B, H, W, C, ksize, _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("slide_attn_oracle_dwconv: invalid arguments")
    return out


def _dense_attention(qv, keys, vals, bias_h):
    """Eq. 2 for one query vector and its gathered keys/values ([n,d] each)."""
    d = qv.shape[0]
    l = keys @ qv / np.sqrt(float(d))
    if bias_h is not None:
        l = l + bias_h
    e = np.exp(l - l.max())
    a = e / e.sum()
    return a @ vals


def im2col_local_attention(q, k, v, ksize, bias=None):
    """Column view (Eq. 4-7): gather each query's window, then attend over it.

    The window of query (i,j) holds K[i+u, j+v] for u,v in [-r,r] in row-major
    (u,v) order, zero where it leaves the map (Fig. 2).  Fixed-shift case only.
    """
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    B, H, W, heads, d = q.shape
    r = ksize // 2
    out = np.zeros_like(q)
    for b in range(B):
        for i in range(H):
            for j in range(W):
                for h in range(heads):
                    col_k, col_v = [], []
                    for u in range(-r, r + 1):
                        for vv in range(-r, r + 1):
                            ii, jj = i + u, j + vv
                            inside = 0 <= ii < H and 0 <= jj < W
                            col_k.append(k[b, ii, jj, h] if inside else np.zeros(d))
                            col_v.append(v[b, ii, jj, h] if inside else np.zeros(d))
                    out[b, i, j, h] = _dense_attention(
                        q[b, i, j, h], np.stack(col_k), np.stack(col_v),
                        None if bias is None else np.asarray(bias, dtype=np.float64)[h])
    return out


def _conv_path(f, w, ksize):
    """One depthwise path (Eq. 12): f [B,H,W,C], w [C,k2,k2] -> [B,H,W,k2,C]."""
    B, H, W, C = f.shape
    r, k2 = ksize // 2, ksize * ksize
    fp = np.zeros((B, H + 2 * r, W + 2 * r, C))
    fp[:, r:r + H, r:r + W] = f
    out = np.zeros((B, H, W, k2, C))
    for s in range(k2):
        for p in range(ksize):
            for q_ in range(ksize):
                out[:, :, :, s, :] += w[:, s, p * ksize + q_] * fp[:, p:p + H, q_:q_ + W, :]
    return out


def two_path_forward(q, k, v, shift_w, learned_wk, learned_wv, ksize, bias=None):
    """Fig. 4 (1): keys/values = fixed-shift conv + learned conv, then Eq. 2."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    E, Dk, Dv = (np.asarray(a, dtype=np.float64) for a in (shift_w, learned_wk, learned_wv))
    B, H, W, heads, d = q.shape
    C = heads * d
    Ks = _conv_path(k.reshape(B, H, W, C), E, ksize) + _conv_path(k.reshape(B, H, W, C), Dk, ksize)
    Vs = _conv_path(v.reshape(B, H, W, C), E, ksize) + _conv_path(v.reshape(B, H, W, C), Dv, ksize)
    out = np.zeros_like(q)
    for b in range(B):
        for i in range(H):
            for j in range(W):
                for h in range(heads):
                    sl = slice(h * d, (h + 1) * d)
                    out[b, i, j, h] = _dense_attention(
                        q[b, i, j, h], Ks[b, i, j][:, sl], Vs[b, i, j][:, sl],
                        None if bias is None else np.asarray(bias, dtype=np.float64)[h])
    return out
