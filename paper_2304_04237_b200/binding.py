"""ctypes binding of libslide_attn.so: the same entry points as include/slide_attn.h.

Argument marshalling only -- every step of the forward runs in the library's CUDA kernels.
PyTorch appears here for device memory and streams alone.  There is no fallback: if the
library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslide_attn.so")

F32, BF16 = 0, 1
VARIANT_AUTO, VARIANT_DIRECT, VARIANT_MMA, VARIANT_UMMA_TS, VARIANT_STRIP, VARIANT_TILE, VARIANT_MMA_WIDE = 0, 1, 2, 5, 6, 8, 9
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ALLOC, ERR_CUDA, ERR_ARCH, ERR_TIMEOUT = range(8)
ERR_TOO_LARGE = 8
ERR_NOT_FIXED_SHIFT = 9

EXPORTS = ("slide_attn_create", "slide_attn_forward", "slide_attn_forward_host", "slide_attn_backward",
           "slide_attn_forward_noalloc", "slide_attn_project", "slide_attn_block_forward",
           "slide_attn_set_variant", "slide_attn_get_variant", "slide_attn_launches_per_forward",
           "slide_attn_set_fixed_shift", "slide_attn_detect_fixed_shift",
           "slide_attn_profile_begin", "slide_attn_profile_end",
           "slide_attn_query_status", "slide_attn_destroy", "slide_attn_status_string")

_lib = None


class SlideAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {slide_attn_status_string(status)} (status {status})")


def load() -> ctypes.CDLL:
    """Loads the shared library; raises if it is missing (build it with
    `python -m paper_2304_04237_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build the CUDA library first "
                               "(python -m paper_2304_04237_b200.build); there is no fallback path")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i = ctypes.c_void_p, ctypes.c_int
        lib.slide_attn_create.argtypes = [ctypes.POINTER(vp), i, i, i, i, i, i, i, i]
        lib.slide_attn_forward.argtypes = [vp] * 9
        lib.slide_attn_forward_host.argtypes = [vp] * 9
        lib.slide_attn_backward.argtypes = [vp] * 15
        lib.slide_attn_forward_noalloc.argtypes = [vp] * 7 + [i] * 7 + [vp]
        lib.slide_attn_project.argtypes = [vp, vp, vp, i, vp, vp, vp, vp]
        lib.slide_attn_block_forward.argtypes = [vp] * 9
        lib.slide_attn_set_variant.argtypes = [vp, i]
        lib.slide_attn_get_variant.argtypes = [vp, ctypes.POINTER(i)]
        lib.slide_attn_set_fixed_shift.argtypes = [vp, i]
        lib.slide_attn_detect_fixed_shift.argtypes = [vp, vp, vp, ctypes.POINTER(i), vp]
        lib.slide_attn_launches_per_forward.argtypes = [vp, ctypes.POINTER(i)]
        lib.slide_attn_profile_begin.argtypes = [vp]
        lib.slide_attn_profile_end.argtypes = [vp, ctypes.POINTER(ctypes.c_double),
                                               ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i)]
        lib.slide_attn_query_status.argtypes = [vp, vp]
        lib.slide_attn_destroy.argtypes = [vp]
        lib.slide_attn_status_string.argtypes = [i]
        lib.slide_attn_status_string.restype = ctypes.c_char_p
        for name in EXPORTS[:-1]:
            getattr(lib, name).restype = i
        _lib = lib
    return _lib


def slide_attn_status_string(status: int) -> str:
    return load().slide_attn_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise SlideAttnError(status, where)


def slide_attn_create(B, H, W, heads, head_dim, ksize, dtype, has_bias) -> int:
    """Returns the context handle (an integer address).  dtype: F32 / BF16 or a torch dtype."""
    if isinstance(dtype, torch.dtype):
        dtype = {torch.float32: F32, torch.bfloat16: BF16}[dtype]
    h = ctypes.c_void_p()
    _check(load().slide_attn_create(ctypes.byref(h), B, H, W, heads, head_dim, ksize, int(dtype),
                                    int(bool(has_bias))), "slide_attn_create")
    return h.value


def _dev_ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("slide_attn_forward takes contiguous CUDA tensors")
    return t.data_ptr()


def _host_ptr(t):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("slide_attn_forward_host takes contiguous CPU tensors")
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def slide_attn_forward(ctx, q, k, v, wk, wv, bias, out, stream=None) -> None:
    """Device tensors in, result written to `out`; asynchronous on `stream`
    (default: torch's current stream)."""
    _check(load().slide_attn_forward(ctx, *map(_dev_ptr, (q, k, v, wk, wv, bias, out)),
                                     _stream_ptr(stream)), "slide_attn_forward")


def slide_attn_backward(ctx, q, k, v, wk, wv, bias, dout, dq, dk, dv, dwk, dwv, dbias, stream=None) -> None:
    """Gradients of the forward's inputs for dout = d(loss)/d(out); device tensors, asynchronous on
    `stream`.  dq, dk, dv: shape and dtype of q; dwk, dwv: float32 like wk; dbias: float32 like bias or None."""
    _check(load().slide_attn_backward(ctx, *map(_dev_ptr, (q, k, v, wk, wv, bias, dout, dq, dk, dv, dwk, dwv, dbias)),
                                      _stream_ptr(stream)), "slide_attn_backward")


def slide_attn_project(ctx, x, w, ys, stream=None) -> None:
    """Eq. 1 / Eq. 3: ys[i] = x w[i] over the tokens of the context's shape.  x and every ys[i]: bf16 device
    tensors [B, H, W, C]; w: float32 device tensor [len(ys), C, C] (input channel, output channel)."""
    ys = list(ys)
    ptrs = [_dev_ptr(y) for y in ys] + [None] * (3 - len(ys))
    _check(load().slide_attn_project(ctx, _dev_ptr(x), _dev_ptr(w), len(ys), *ptrs, _stream_ptr(stream)),
           "slide_attn_project")


def slide_attn_block_forward(ctx, x, w_qkv, w_o, wk, wv, bias, out, stream=None) -> None:
    """A whole block: projections (Eq. 1, w_qkv float32 [3, C, C]), the local attention, output projection
    (Eq. 3, w_o float32 [C, C]); x and out bf16 device tensors [B, H, W, C]."""
    _check(load().slide_attn_block_forward(ctx, *map(_dev_ptr, (x, w_qkv, w_o, wk, wv, bias, out)),
                                           _stream_ptr(stream)), "slide_attn_block_forward")


def slide_attn_forward_host(ctx, q, k, v, wk, wv, bias, out, stream=None) -> None:
    """CPU tensors in and out (pinned for best speed); returns when `out` is filled."""
    _check(load().slide_attn_forward_host(ctx, *map(_host_ptr, (q, k, v, wk, wv, bias, out)),
                                          _stream_ptr(stream)), "slide_attn_forward_host")


def slide_attn_forward_noalloc(q, k, v, wk, wv, bias, out, ksize, stream=None) -> None:
    """Forward for callers that must not allocate device memory: no context, the library's
    fixed scratch is used instead (bf16, head_dim 32, ksize 3, at most 16 heads).  The shape is
    taken from `q` ([B, H, W, heads, head_dim]).  Calls that overlap on the GPU race on the
    shared scratch; keep them on one stream."""
    B, H, W, heads, head_dim = q.shape
    dtype = {torch.float32: F32, torch.bfloat16: BF16}[q.dtype]
    _check(load().slide_attn_forward_noalloc(*map(_dev_ptr, (q, k, v, wk, wv, bias, out)),
                                             B, H, W, heads, head_dim, int(ksize), dtype,
                                             _stream_ptr(stream)), "slide_attn_forward_noalloc")


def slide_attn_set_variant(ctx, variant: int) -> None:
    _check(load().slide_attn_set_variant(ctx, int(variant)), "slide_attn_set_variant")


def slide_attn_set_fixed_shift(ctx, enable: bool) -> None:
    """Declares that later forwards get exactly the one-hot shift kernels as wk and wv (checked on
    the device in every forward); they then run the fixed-shift kernel."""
    _check(load().slide_attn_set_fixed_shift(ctx, int(bool(enable))), "slide_attn_set_fixed_shift")


def slide_attn_detect_fixed_shift(ctx, wk, wv, stream=None) -> bool:
    """True if the device tensors wk and wv are exactly the one-hot shift kernels (synchronises)."""
    r = ctypes.c_int()
    _check(load().slide_attn_detect_fixed_shift(ctx, _dev_ptr(wk), _dev_ptr(wv), ctypes.byref(r), _stream_ptr(stream)),
           "slide_attn_detect_fixed_shift")
    return bool(r.value)


def slide_attn_get_variant(ctx) -> int:
    v = ctypes.c_int()
    _check(load().slide_attn_get_variant(ctx, ctypes.byref(v)), "slide_attn_get_variant")
    return v.value


def slide_attn_launches_per_forward(ctx) -> int:
    n = ctypes.c_int()
    _check(load().slide_attn_launches_per_forward(ctx, ctypes.byref(n)), "slide_attn_launches_per_forward")
    return n.value


def slide_attn_profile_begin(ctx) -> None:
    _check(load().slide_attn_profile_begin(ctx), "slide_attn_profile_begin")


def slide_attn_profile_end(ctx):
    """Returns (mean ms per forward, mean ms of the main kernel, forwards averaged)."""
    f, m, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    _check(load().slide_attn_profile_end(ctx, ctypes.byref(f), ctypes.byref(m), ctypes.byref(n)),
           "slide_attn_profile_end")
    return f.value, m.value, n.value


def slide_attn_query_status(ctx, stream=None) -> int:
    """Synchronises the stream; returns OK or ERR_TIMEOUT (does not raise on timeout)."""
    st = load().slide_attn_query_status(ctx, _stream_ptr(stream))
    if st not in (OK, ERR_TIMEOUT, ERR_NOT_FIXED_SHIFT):
        raise SlideAttnError(st, "slide_attn_query_status")
    return st


def slide_attn_destroy(ctx) -> None:
    _check(load().slide_attn_destroy(ctx), "slide_attn_destroy")
