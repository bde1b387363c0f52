"""Helpers shared by the GPU parity tests: uploading seeded host inputs, calling the
library through its C ABI, and the error criterion."""
import numpy as np
import torch

import paper_2304_04237_b200 as sa

TOL = {"f32": 1e-4, "bf16": 2e-2}     # |gpu - ref| <= tol * max(1, |ref|)
TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}
VARIANTS = {"direct": sa.VARIANT_DIRECT, "mma": sa.VARIANT_MMA, "umma_ts": sa.VARIANT_UMMA_TS, "strip": sa.VARIANT_STRIP,
            "tile": sa.VARIANT_TILE, "mma_wide": sa.VARIANT_MMA_WIDE}


def to_device(x, dtype):
    """Host float32 arrays (already holding storage-dtype values) -> CUDA tensors."""
    td = TORCH_DTYPE[dtype]
    dev = {}
    for n in ("q", "k", "v"):
        dev[n] = torch.from_numpy(x[n]).to(td).cuda().contiguous()
    for n in ("wk", "wv"):
        dev[n] = torch.from_numpy(x[n]).cuda().contiguous()
    dev["bias"] = None if x["bias"] is None else torch.from_numpy(x["bias"]).cuda().contiguous()
    return dev


def gpu_forward(x, ksize, dtype, variant=None, out=None):
    """Runs the library on host inputs `x`; returns out as float64 numpy [B,H,W,heads,d].
    Raises sa.SlideAttnError(ERR_UNSUPPORTED) if the variant cannot run the shape."""
    B, H, W, heads, d = x["q"].shape
    dev = to_device(x, dtype)
    ctx = sa.slide_attn_create(B, H, W, heads, d, ksize, TORCH_DTYPE[dtype], x["bias"] is not None)
    try:
        if variant is not None:
            sa.slide_attn_set_variant(ctx, VARIANTS[variant] if isinstance(variant, str) else variant)
        if out is None:
            out = torch.full_like(dev["q"], float("nan"))
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
        torch.cuda.synchronize()
        assert sa.slide_attn_query_status(ctx) == sa.OK
    finally:
        sa.slide_attn_destroy(ctx)
    return out.float().cpu().numpy().astype(np.float64)


def assert_close(got, ref, dtype, what=""):
    tol = TOL[dtype]
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref) / np.maximum(1.0, np.abs(ref))
    worst = float(err.max()) if err.size else 0.0
    assert worst <= tol, f"{what}: max err {worst:.3e} > {tol:g} at {np.unravel_index(err.argmax(), err.shape)}"
    return worst
