"""GPU parity of the fixed-shift fast path (one-hot depthwise kernels: plain k x k local attention,
Sec. 4.2) against the CPU oracle given the same one-hot weights, for every supported window size and
both dtypes; bit-exact index / halo / padding checks with integer inputs on the key and on the value
side; and the device-side check of the caller's declaration."""
import zlib

import numpy as np
import pytest
import torch

import oracle
import paper_2304_04237_b200 as sa
from paper_2304_04237_b200 import synth

from util import TORCH_DTYPE, assert_close, to_device

pytestmark = pytest.mark.gpu


def shift_forward(x, k, dtype, expect=sa.OK):
    """Forward in fixed-shift mode; returns out as float64 numpy."""
    B, H, W, heads, d = x["q"].shape
    dev = to_device(x, dtype)
    ctx = sa.slide_attn_create(B, H, W, heads, d, k, TORCH_DTYPE[dtype], x["bias"] is not None)
    try:
        sa.slide_attn_set_fixed_shift(ctx, True)
        assert sa.slide_attn_launches_per_forward(ctx) == 2
        out = torch.full_like(dev["q"], float("nan"))
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
        torch.cuda.synchronize()
        assert sa.slide_attn_query_status(ctx) == expect
    finally:
        sa.slide_attn_destroy(ctx)
    return out.float().cpu().numpy().astype(np.float64)


SHAPES = [  # B, H, W, heads, k
    (2, 14, 14, 2, 3), (1, 17, 13, 3, 3), (2, 1, 1, 1, 3), (1, 2, 2, 1, 3), (1, 33, 47, 2, 3), (3, 9, 70, 1, 3),
    (1, 3, 5, 2, 5), (1, 1, 19, 1, 5), (2, 13, 37, 2, 5), (1, 5, 2, 1, 7), (1, 17, 34, 1, 7), (1, 9, 11, 2, 9),
    (1, 3, 3, 1, 9), (1, 20, 41, 3, 9), (3, 7, 5, 2, 1), (2, 28, 42, 6, 3),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_fixed_shift_matches_oracle(shape, dtype):
    B, H, W, heads, k = shape
    seed = zlib.crc32(repr(shape).encode()) & 0xFFFFFF
    x = synth.make_inputs(B, H, W, heads, 32, k, dtype, 0.0, 0.3, True, seed=seed)   # sigma_w = 0: one-hot weights
    assert np.array_equal(x["wk"], synth.one_hot_weights(heads * 32, k))
    ref = oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k)
    assert_close(shift_forward(x, k, dtype), ref, dtype, f"fixed shift {shape} {dtype}")


@pytest.mark.parametrize("name", ["c2", "c3_k5", "c5_k7", "c5_k9", "c5_f32"])
def test_fixed_shift_full_size_every_element(name):
    """The bench shapes with one-hot weights, every element against the oracle."""
    cfg = dict(synth.CONFIGS[name])
    cfg["sigma_w"] = 0.0
    if name in ("c2", "c3_k5"):
        cfg["B"] = 8                       # the oracle's time; the tiling does not depend on the batch
    x = synth.make_inputs(**cfg)
    ref = oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], cfg["ksize"])
    assert_close(shift_forward(x, cfg["ksize"], cfg["dtype"]), ref, cfg["dtype"], f"fixed shift {name}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,W,k", [(28, 42, 3), (13, 17, 3), (2, 2, 3), (13, 37, 5), (3, 2, 5), (9, 40, 7), (5, 9, 9),
                                   (17, 33, 9), (4, 4, 1)])
def test_value_index_logic_bit_exact(H, W, k, dtype):
    """q = 0 and a bias of 0 on one slot, -1000 on the others: the attention is exactly one-hot, so
    out must equal v read at that slot's offset (zero outside the map), compared with ==."""
    B, heads, d, r, k2 = 2, 2, 32, k // 2, k * k
    rng = np.random.default_rng(H * 100 + W + k)
    v = rng.integers(0, 256, size=(B, H, W, heads, d)).astype(np.float32)
    kk = rng.integers(-3, 4, size=v.shape).astype(np.float32)
    E = synth.one_hot_weights(heads * d, k)
    for s0 in sorted({0, k2 // 2, k2 - 1, k - 1, k2 - k, (k2 // 2 + 1) % k2}):
        s1 = (s0 * 7 + 3) % k2
        bias = np.full((heads, k2), -1000.0, np.float32)
        bias[0, s0] = 0
        bias[1, s1] = 0
        got = shift_forward(dict(q=np.zeros_like(v), k=kk, v=v, wk=E, wv=E, bias=bias), k, dtype)
        for h, s in ((0, s0), (1, s1)):
            u, vv = s // k - r, s % k - r
            want = np.zeros_like(v[:, :, :, h])
            ys, xs = slice(max(0, -u), min(H, H - u)), slice(max(0, -vv), min(W, W - vv))
            yd, xd = slice(max(0, u), min(H, H + u)), slice(max(0, vv), min(W, W + vv))
            want[:, ys, xs] = v[:, yd, xd, h]
            assert np.array_equal(got[:, :, :, h], want.astype(np.float64)), (s, h)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,W,k", [(28, 42, 3), (13, 17, 3), (2, 2, 3), (1, 1, 3), (1, 7, 3), (33, 47, 3),
                                   (13, 37, 5), (3, 2, 5), (9, 40, 7), (5, 9, 9), (17, 33, 9)])
def test_key_index_logic_bit_exact(H, W, k, dtype):
    """q is 64 on one channel per head; k on that channel is 16 * (1 + k * (i mod k) + (j mod k)): the
    in-map neighbours of a pixel carry distinct integer keys (exact in bf16), padded slots carry 0, and
    two logits differ by at least 64 * 16 / sqrt(32) = 181, so every softmax weight but one underflows
    to exactly 0 and out must equal v at the in-map neighbour with the largest key, compared with ==."""
    B, heads, d, r = 2, 2, 32, k // 2
    rng = np.random.default_rng(H * 131 + W * 7 + k)
    v = rng.integers(0, 256, size=(B, H, W, heads, d)).astype(np.float32)
    code = (16 * (1 + k * (np.arange(H)[:, None] % k) + (np.arange(W)[None, :] % k))).astype(np.float32)
    q, kk, want = np.zeros_like(v), np.zeros_like(v), np.zeros_like(v)
    padded = np.zeros((H + 2 * r, W + 2 * r), np.float32)
    padded[r:r + H, r:r + W] = code
    for h in range(heads):
        ch = (7 * h + 3) % d
        q[:, :, :, h, ch] = 64.0
        kk[:, :, :, h, ch] = code[None]
    for i in range(H):
        for j in range(W):
            win = padded[i:i + k, j:j + k]
            u, vv = np.unravel_index(int(win.argmax()), win.shape)
            want[:, i, j] = v[:, i + u - r, j + vv - r]
    E = synth.one_hot_weights(heads * d, k)
    got = shift_forward(dict(q=q, k=kk, v=v, wk=E, wv=E, bias=None), k, dtype)
    assert np.array_equal(got, want.astype(np.float64))


def test_declaration_is_checked_on_the_device():
    """A weight that is not one-hot: the detection helper says so, and a forward in fixed-shift mode
    reports it through the status word; with the one-hot kernels both are quiet."""
    B, H, W, heads, k = 1, 9, 12, 2, 3
    x = synth.make_inputs(B, H, W, heads, 32, k, "bf16", 0.0, 0.1, True, seed=5)
    dev = to_device(x, "bf16")
    ctx = sa.slide_attn_create(B, H, W, heads, 32, k, torch.bfloat16, True)
    try:
        assert sa.slide_attn_detect_fixed_shift(ctx, dev["wk"], dev["wv"]) is True
        bad = dev["wv"].clone()
        bad[37, 4, 5] = 1e-3
        assert sa.slide_attn_detect_fixed_shift(ctx, dev["wk"], bad) is False
        assert sa.slide_attn_query_status(ctx) == sa.OK          # the helper leaves the status word alone
        sa.slide_attn_set_fixed_shift(ctx, True)
        out = torch.empty_like(dev["q"])
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], bad, dev["bias"], out)
        assert sa.slide_attn_query_status(ctx) == sa.ERR_NOT_FIXED_SHIFT
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
        assert sa.slide_attn_query_status(ctx) == sa.OK
        sa.slide_attn_set_fixed_shift(ctx, False)
        assert sa.slide_attn_launches_per_forward(ctx) in (1, 2)
    finally:
        sa.slide_attn_destroy(ctx)


def test_unsupported_shapes_keep_the_mode_off():
    ctx = sa.slide_attn_create(1, 4, 4, 1, 16, 3, torch.float32, False)      # head_dim 16
    try:
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_set_fixed_shift(ctx, True)
        assert e.value.status == sa.ERR_UNSUPPORTED
    finally:
        sa.slide_attn_destroy(ctx)
