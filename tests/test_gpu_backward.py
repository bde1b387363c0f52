"""GPU parity of the backward pass (slide_attn_backward through the C ABI) against the backward oracle,
which is itself pinned by finite differences of the forward oracle (tests/test_oracle_backward.py)."""
import zlib

import numpy as np
import pytest
import torch

import paper_2304_04237_b200 as sa
from oracle import backward as ob
from paper_2304_04237_b200 import synth

from util import TOL, TORCH_DTYPE, to_device

pytestmark = pytest.mark.gpu


def gpu_backward(x, dout, k, dtype, repeat=1):
    B, H, W, heads, d = x["q"].shape
    dev = to_device(x, dtype)
    td = TORCH_DTYPE[dtype]
    g = torch.from_numpy(dout).to(td).cuda().contiguous()
    outs = []
    ctx = sa.slide_attn_create(B, H, W, heads, d, k, td, x["bias"] is not None)
    try:
        for _ in range(repeat):
            dq, dk, dv = (torch.full_like(dev["q"], float("nan")) for _ in range(3))
            dwk, dwv = (torch.full_like(dev["wk"], float("nan")) for _ in range(2))
            dbias = None if dev["bias"] is None else torch.full_like(dev["bias"], float("nan"))
            sa.slide_attn_backward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], g,
                                   dq, dk, dv, dwk, dwv, dbias)
            torch.cuda.synchronize()
            assert sa.slide_attn_query_status(ctx) == sa.OK
            outs.append(dict(dq=dq, dk=dk, dv=dv, dwk=dwk, dwv=dwv, dbias=dbias))
    finally:
        sa.slide_attn_destroy(ctx)
    f64 = lambda t: None if t is None else t.float().cpu().numpy().astype(np.float64)
    return [{n: f64(t) for n, t in o.items()} for o in outs]


def check(got, ref, dtype, what):
    for n in ("dq", "dk", "dv"):
        assert np.isfinite(got[n]).all(), (what, n)
        err = np.abs(got[n] - ref[n]) / np.maximum(1.0, np.abs(ref[n]))
        assert err.max() <= TOL[dtype], f"{what} {n}: {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    for n in ("dwk", "dwv", "dbias"):           # sums over all pixels: relative to the largest entry
        if ref[n] is None:
            assert got[n] is None
            continue
        assert np.isfinite(got[n]).all(), (what, n)
        err = np.abs(got[n] - ref[n]).max() / max(1.0, np.abs(ref[n]).max())
        assert err <= 5e-4, f"{what} {n}: {err:.3e}"


def inputs(shape, dtype, bias=True, sigma_w=0.05):
    B, H, W, heads, k = shape
    seed = zlib.crc32(repr(shape).encode()) & 0xFFFFFF
    x = synth.make_inputs(B, H, W, heads, 32, k, dtype, sigma_w, 0.3, bias, seed=seed)
    dout = np.random.default_rng(seed).normal(size=x["q"].shape).astype(np.float32)
    if dtype == "bf16":
        dout = torch.from_numpy(dout).to(torch.bfloat16).float().numpy()      # the stored values
    return x, dout


SHAPES = [(1, 4, 8, 1, 3), (2, 14, 14, 2, 3), (1, 17, 13, 3, 3), (2, 1, 1, 1, 3), (1, 2, 2, 1, 3), (1, 9, 70, 2, 3),
          (3, 7, 5, 2, 1), (1, 33, 47, 2, 3), (2, 28, 42, 6, 3)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_backward_matches_oracle(shape, dtype):
    x, dout = inputs(shape, dtype)
    ref = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], shape[4], dout)
    got = gpu_backward(x, dout, shape[4], dtype)[0]
    check(got, ref, dtype, f"{shape} {dtype}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_backward_no_bias_dense_weights_and_repeat(dtype):
    """Weights far from one-hot, no bias; a second call on the same context overwrites (does not
    accumulate into) every gradient."""
    shape = (2, 15, 18, 2, 3)
    x, dout = inputs(shape, dtype, bias=False, sigma_w=0.4)
    ref = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], None, 3, dout)
    a, b = gpu_backward(x, dout, 3, dtype, repeat=2)
    check(a, ref, dtype, "dense first")
    check(b, ref, dtype, "dense second")
    for n in ("dq", "dk", "dv"):
        assert np.array_equal(a[n], b[n])           # no atomics on these: bit-identical


def test_backward_stage_shape_sample():
    """Four images of the bench shape (56 x 56, 2 heads), bf16."""
    x, dout = inputs((4, 56, 56, 2, 3), "bf16", sigma_w=0.02)
    ref = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], 3, dout)
    check(gpu_backward(x, dout, 3, "bf16")[0], ref, "bf16", "4x56x56x2")


def test_backward_argument_errors():
    ctx = sa.slide_attn_create(1, 4, 4, 1, 32, 5, torch.float32, False)          # k = 5: no backward kernel
    try:
        t = torch.zeros(1, 4, 4, 1, 32, device="cuda")
        w = torch.zeros(32, 25, 25, device="cuda")
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_backward(ctx, t, t.clone(), t.clone(), w, w.clone(), None, t.clone(), t.clone(), t.clone(), t.clone(),
                                   w.clone(), w.clone(), None)
        assert e.value.status == sa.ERR_UNSUPPORTED
    finally:
        sa.slide_attn_destroy(ctx)
    ctx = sa.slide_attn_create(1, 4, 4, 1, 32, 3, torch.float32, False)
    try:
        t = torch.zeros(1, 4, 4, 1, 32, device="cuda")
        w = torch.zeros(32, 9, 9, device="cuda")
        with pytest.raises(sa.SlideAttnError) as e:                              # dq aliases q
            sa.slide_attn_backward(ctx, t, t.clone(), t.clone(), w, w.clone(), None, t.clone(), t, t.clone(), t.clone(),
                                   w.clone(), w.clone(), None)
        assert e.value.status == sa.ERR_INVALID_ARG
    finally:
        sa.slide_attn_destroy(ctx)
