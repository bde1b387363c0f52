"""GPU parity of the block entry points (slide_attn_project, slide_attn_block_forward: Eq. 1 - 3 around the
local attention) through the C ABI against the block oracle (oracle/block.py, pinned by
tests/test_oracle_block.py)."""
import zlib

import numpy as np
import pytest
import torch

import paper_2304_04237_b200 as sa
from oracle import block as ob
from paper_2304_04237_b200 import synth

from util import TOL

pytestmark = pytest.mark.gpu


def bf16_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda().contiguous()


def f32_dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().contiguous()


def head_split(C):
    """(heads, head_dim) of a context with C channels."""
    return (C // 32, 32) if C % 32 == 0 else (C // 16, 16)


def gpu_project(x, w, shape):
    B, H, W, C = shape
    heads, d = head_split(C)
    xd, wd = bf16_dev(x), f32_dev(w)
    ys = [torch.full((B, H, W, C), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.shape[0])]
    ctx = sa.slide_attn_create(B, H, W, heads, d, 3, torch.bfloat16, False)
    try:
        sa.slide_attn_project(ctx, xd, wd, ys)
        torch.cuda.synchronize()
        assert sa.slide_attn_query_status(ctx) == sa.OK
    finally:
        sa.slide_attn_destroy(ctx)
    return [y.float().cpu().numpy().astype(np.float64) for y in ys]


@pytest.mark.parametrize("shape", [(1, 1, 1, 16), (1, 3, 5, 32), (2, 9, 15, 64), (1, 13, 21, 96), (1, 17, 8, 192), (3, 7, 11, 256),
                                   (1, 16, 16, 48), (1, 40, 40, 224)], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("nmat", [1, 2, 3])
def test_project_is_bit_exact_on_small_integers(shape, nmat):
    """Integer tokens and sparse integer weights (two taps per output channel): every sum is a small integer, exact
    in bf16, so each output must equal the integer result bit for bit -- row / channel / matrix indexing, the
    chunking of wide outputs and the ragged last row tile."""
    B, H, W, C = shape
    rng = np.random.default_rng(zlib.crc32(repr((shape, nmat)).encode()))
    x = rng.integers(-3, 4, size=(B, H, W, C)).astype(np.float32)
    w = np.zeros((nmat, C, C), dtype=np.float32)
    for m in range(nmat):
        for o in range(C):
            taps = rng.choice(C, size=2, replace=False)
            w[m, taps, o] = rng.choice([-2.0, -1.0, 1.0, 2.0], size=2)
    got = gpu_project(x, w, shape)
    for m in range(nmat):
        want = x.astype(np.float64) @ w[m].astype(np.float64)
        np.testing.assert_array_equal(got[m], want)


@pytest.mark.parametrize("shape", [(2, 14, 14, 64), (1, 33, 47, 96), (1, 28, 28, 192), (1, 20, 20, 256),
                                   # more than two row tiles per CTA, for every number of accumulator slots
                                   (1, 210, 200, 32), (1, 200, 200, 96), (1, 200, 200, 128), (1, 200, 200, 192), (1, 199, 200, 256)],
                         ids=lambda s: "x".join(map(str, s)))
def test_project_random_matches_double(shape):
    B, H, W, C = shape
    rng = np.random.default_rng(zlib.crc32(repr(shape).encode()))
    x = ob.round_bf16(rng.normal(size=(B, H, W, C)))
    w = (rng.normal(size=(3, C, C)) / np.sqrt(C)).astype(np.float32)
    got = gpu_project(x, w, shape)
    for m in range(3):
        want = ob.project(x, ob.round_bf16(w[m]))              # the kernel's weights are the bf16 values
        err = np.abs(got[m] - want) / np.maximum(1.0, np.abs(want))
        assert err.max() <= 2.0 ** -8 + 1e-5, (m, err.max())     # one rounding to bf16 of an fp32-accumulated sum


def block_inputs(shape, seed_extra=0, sigma_w=0.05):
    B, H, W, heads, k = shape
    C = heads * 32
    seed = (zlib.crc32(repr(shape).encode()) + seed_extra) & 0xFFFFFF
    a = synth.make_inputs(B, H, W, heads, 32, k, "bf16", sigma_w, 0.3, True, seed=seed)
    rng = np.random.default_rng(seed)
    p = dict(x=ob.round_bf16(rng.normal(size=(B, H, W, C))).astype(np.float32), wk=a["wk"], wv=a["wv"], bias=a["bias"])
    p["w_qkv"] = (rng.normal(size=(3, C, C)) / np.sqrt(C)).astype(np.float32)
    p["w_o"] = (rng.normal(size=(C, C)) / np.sqrt(C)).astype(np.float32)
    return p


def oracle_block(p, k, heads):
    # the product's weights are the bf16 values of the fp32 matrices
    wq, wk_, wv_ = (ob.round_bf16(p["w_qkv"][i]) for i in range(3))
    return ob.block_forward(p["x"], wq, wk_, wv_, ob.round_bf16(p["w_o"]), p["wk"], p["wv"], p["bias"], k, heads, storage="bf16")


def gpu_block(p, shape, repeat=1, fixed_shift=False):
    B, H, W, heads, k = shape
    C = heads * 32
    dev = dict(x=bf16_dev(p["x"]), w_qkv=f32_dev(p["w_qkv"]), w_o=f32_dev(p["w_o"]), wk=f32_dev(p["wk"]), wv=f32_dev(p["wv"]),
               bias=f32_dev(p["bias"]))
    outs = []
    ctx = sa.slide_attn_create(B, H, W, heads, 32, k, torch.bfloat16, p["bias"] is not None)
    try:
        if fixed_shift:
            sa.slide_attn_set_fixed_shift(ctx, True)
        for _ in range(repeat):
            out = torch.full((B, H, W, C), float("nan"), dtype=torch.bfloat16, device="cuda")
            sa.slide_attn_block_forward(ctx, dev["x"], dev["w_qkv"], dev["w_o"], dev["wk"], dev["wv"], dev["bias"], out)
            torch.cuda.synchronize()
            assert sa.slide_attn_query_status(ctx) == sa.OK
            outs.append(out.float().cpu().numpy().astype(np.float64))
    finally:
        sa.slide_attn_destroy(ctx)
    return outs


def assert_block_close(got, ref, what):
    assert np.isfinite(got).all(), what
    err = np.abs(got - ref) / np.maximum(1.0, np.abs(ref))
    assert err.max() <= TOL["bf16"], f"{what}: {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    return float(err.max())


SHAPES = [(1, 8, 8, 1, 3), (2, 14, 14, 2, 3), (1, 17, 13, 3, 3), (1, 9, 70, 2, 3), (2, 28, 42, 6, 3), (1, 12, 12, 8, 3),
          (1, 10, 10, 2, 5), (1, 6, 6, 2, 1), (1, 1, 1, 1, 3), (3, 5, 130, 2, 3)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_block_forward_matches_oracle(shape):
    p = block_inputs(shape)
    ref = oracle_block(p, shape[4], shape[3])
    got = gpu_block(p, shape, repeat=2)
    assert_block_close(got[0], ref, f"{shape}")
    np.testing.assert_array_equal(got[0], got[1])                   # a second call on the same context: same bits


def test_block_forward_fixed_shift_mode():
    shape = (2, 14, 14, 2, 3)
    p = block_inputs(shape, sigma_w=0.0)
    ref = oracle_block(p, 3, 2)
    assert_block_close(gpu_block(p, shape, fixed_shift=True)[0], ref, "fixed shift")


def test_block_forward_full_size_every_element():
    """The bench workload's shape (B = 64, 56 x 56, 2 heads x 32, k = 3): every element against the oracle."""
    shape = (64, 56, 56, 2, 3)
    p = block_inputs(shape, sigma_w=0.02)
    ref = oracle_block(p, 3, 2)
    worst = assert_block_close(gpu_block(p, shape)[0], ref, "c2-sized block")
    print(f"block c2: worst error {worst:.3e}")


def test_block_argument_errors():
    ctx = sa.slide_attn_create(1, 4, 4, 1, 32, 3, torch.bfloat16, False)
    x = torch.zeros((1, 4, 4, 32), dtype=torch.bfloat16, device="cuda")
    w3 = torch.zeros((3, 32, 32), device="cuda")
    w1 = torch.zeros((32, 32), device="cuda")
    wk = torch.zeros((32, 9, 9), device="cuda")
    try:
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_block_forward(ctx, x, w3, w1, wk, wk, None, x)
        assert e.value.status == sa.ERR_INVALID_ARG                  # out aliases x
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_project(ctx, x, w3, [x])
        assert e.value.status == sa.ERR_INVALID_ARG
        y = torch.zeros_like(x)
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_project(ctx, x, w3, [y, y])
        assert e.value.status == sa.ERR_INVALID_ARG                  # two outputs alias
    finally:
        sa.slide_attn_destroy(ctx)
    ctx = sa.slide_attn_create(1, 4, 4, 1, 32, 3, torch.float32, False)
    try:
        xf = torch.zeros((1, 4, 4, 32), device="cuda")
        with pytest.raises(sa.SlideAttnError) as e:
            sa.slide_attn_block_forward(ctx, xf, w3, w1, wk, wk, None, torch.zeros_like(xf))
        assert e.value.status == sa.ERR_UNSUPPORTED                  # bf16 contexts only
    finally:
        sa.slide_attn_destroy(ctx)
