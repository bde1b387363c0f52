"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Criterion: |gpu - ref| <= tol * max(1, |ref|), tol = 1e-4 (fp32) / 2e-2 (bf16);
index / halo / padding logic is checked bit-exactly with integer-valued inputs."""
import zlib

import numpy as np
import pytest
import torch

import oracle
import paper_2304_04237_b200 as sa
from paper_2304_04237_b200 import synth

from util import TORCH_DTYPE, VARIANTS, assert_close, gpu_forward, to_device

pytestmark = pytest.mark.gpu

ALL_VARIANTS = ["auto", "direct", "strip", "tile", "mma", "mma_wide", "umma_ts"]
PIPELINED = ["umma_ts"]


def ref_forward(x, k):
    return oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k)


def run_variant(x, k, dtype, variant):
    """Output of the variant, or None when it does not support the shape/dtype."""
    try:
        return gpu_forward(x, k, dtype, None if variant == "auto" else variant)
    except sa.SlideAttnError as e:
        if e.status == sa.ERR_UNSUPPORTED and variant != "auto":
            return None
        raise


# ---- the tiny configuration, element by element -----------------------------------------

@pytest.mark.parametrize("variant", ALL_VARIANTS)
def test_tiny_config_full(variant):
    cfg, x = synth.make_config("c1_tiny")
    got = run_variant(x, cfg["ksize"], cfg["dtype"], variant)
    if got is None:
        pytest.skip("variant does not support this shape")
    assert_close(got, ref_forward(x, cfg["ksize"]), cfg["dtype"], "c1_tiny")


# ---- small shapes: several tiles, ragged tails, maps smaller than the window ------------

SMALL = [  # B, H, W, heads, d, k
    (2, 14, 14, 2, 32, 3), (1, 17, 13, 3, 32, 3), (2, 1, 1, 1, 32, 3), (1, 2, 2, 1, 32, 3),
    (1, 3, 5, 2, 32, 5), (1, 1, 19, 1, 32, 5), (2, 13, 17, 2, 32, 5), (1, 5, 2, 1, 32, 7),
    (1, 17, 14, 1, 32, 7), (1, 9, 11, 2, 32, 9), (1, 3, 3, 1, 32, 9), (3, 7, 5, 2, 32, 1),
    (1, 30, 33, 2, 32, 3), (1, 29, 43, 6, 32, 3), (2, 31, 9, 1, 32, 3), (1, 16, 64, 1, 32, 3),
    (1, 6, 7, 2, 8, 3), (1, 5, 6, 1, 64, 3), (1, 4, 9, 2, 16, 5), (1, 5, 5, 1, 40, 3),
    (1, 4, 4, 1, 32, 11), (1, 3, 4, 1, 8, 13), (1, 2, 5, 1, 8, 15),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SMALL, ids=lambda s: "x".join(map(str, s)))
def test_small_shapes_all_variants(shape, dtype):
    B, H, W, heads, d, k = shape
    seed = zlib.crc32(repr(shape).encode()) & 0xFFFFFF
    x = synth.make_inputs(B, H, W, heads, d, k, dtype, 0.05, 0.2, True, seed=seed)
    ref = ref_forward(x, k)
    ran = 0
    for variant in ALL_VARIANTS:
        got = run_variant(x, k, dtype, variant)
        if got is None:
            continue
        ran += 1
        assert_close(got, ref, dtype, f"{shape} {dtype} {variant}")
    assert ran >= 2      # auto and direct always run


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_no_bias_and_dense_weights(dtype):
    """Weights far from one-hot (a general merged kernel) and no bias."""
    B, H, W, heads, d, k = 2, 15, 18, 2, 32, 3
    x = synth.make_inputs(B, H, W, heads, d, k, dtype, 0.4, 0.0, False, seed=77)
    ref = ref_forward(x, k)
    for variant in ALL_VARIANTS:
        got = run_variant(x, k, dtype, variant)
        if got is not None:
            assert_close(got, ref, dtype, f"dense-w {variant}")


# ---- bit-exact index / halo / padding check with integer-valued inputs -------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,W,k", [(28, 42, 3), (13, 17, 3), (2, 2, 3), (13, 17, 5), (3, 2, 5),
                                   (9, 20, 7), (5, 9, 9), (56, 56, 3), (33, 47, 3)])
def test_index_logic_bit_exact(H, W, k, dtype):
    """q = 0 and a bias of 0 on one slot, -1000 on the others make the attention exactly
    one-hot, so with the fixed-shift kernels out must equal v read at that slot's offset
    (zero outside the map) -- compared with ==.  v holds small integers (exact in bf16)."""
    B, heads, d, r, k2 = 2, 2, 32, k // 2, k * k
    rng = np.random.default_rng(H * 100 + W + k)
    v = rng.integers(0, 256, size=(B, H, W, heads, d)).astype(np.float32)
    kk = rng.integers(-3, 4, size=v.shape).astype(np.float32)
    E = synth.one_hot_weights(heads * d, k)
    slots = sorted({0, k2 // 2, k2 - 1, k - 1, k2 - k, (k2 // 2 + 1) % k2})
    for variant in ALL_VARIANTS:
        for s0 in slots:
            s1 = (s0 * 7 + 3) % k2
            bias = np.full((heads, k2), -1000.0, np.float32)
            bias[0, s0] = 0
            bias[1, s1] = 0
            x = dict(q=np.zeros_like(v), k=kk, v=v, wk=E, wv=E, bias=bias)
            got = run_variant(x, k, dtype, variant)
            if got is None:
                break
            for h, s in ((0, s0), (1, s1)):
                u, vv = s // k - r, s % k - r
                want = np.zeros_like(v[:, :, :, h])
                ys, xs = slice(max(0, -u), min(H, H - u)), slice(max(0, -vv), min(W, W - vv))
                yd, xd = slice(max(0, u), min(H, H + u)), slice(max(0, vv), min(W, W + vv))
                want[:, ys, xs] = v[:, yd, xd, h]
                assert np.array_equal(got[:, :, :, h], want.astype(np.float64)), (variant, s, h)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,W,k", [(28, 42, 3), (13, 17, 3), (2, 2, 3), (1, 1, 3), (1, 7, 3), (56, 56, 3),
                                   (33, 47, 3), (13, 17, 5), (3, 2, 5), (9, 20, 7), (5, 9, 9)])
def test_key_index_logic_bit_exact(H, W, k, dtype):
    """The key side of the same check.  q is 64 on one channel per head and 0 elsewhere; k on that
    channel is 16 * (1 + k * (i mod k) + (j mod k)), so the in-map neighbours of a pixel carry
    distinct integer keys (exact in bf16), padded slots carry 0, and two logits differ by at least
    64 * 16 / sqrt(32) = 181: every other softmax weight underflows to exactly 0.  With the
    fixed-shift kernels and no bias, out must equal v at the in-map neighbour with the largest key,
    compared with ==.  A swapped dy/dx, an off-by-one halo origin or a wrong zero fill on the key
    side picks another neighbour."""
    B, heads, d, r = 2, 2, 32, k // 2
    rng = np.random.default_rng(H * 131 + W * 7 + k)
    v = rng.integers(0, 256, size=(B, H, W, heads, d)).astype(np.float32)
    code = (16 * (1 + k * (np.arange(H)[:, None] % k) + (np.arange(W)[None, :] % k))).astype(np.float32)
    q = np.zeros_like(v)
    kk = np.zeros_like(v)
    want = np.zeros_like(v)
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
    x = dict(q=q, k=kk, v=v, wk=E, wv=E, bias=None)
    for variant in ALL_VARIANTS:
        got = run_variant(x, k, dtype, variant)
        if got is None:
            continue
        assert np.array_equal(got, want.astype(np.float64)), (variant, H, W, k)


# ---- full-size configurations, every element, in the launch configuration the bench times ------

def sample_pixels(B, H, W, n, seed):
    """Corners, border runs and tile seams of a few images plus random pixels."""
    rng = np.random.default_rng(seed)
    pts = set()
    for b in {0, B - 1, B // 2}:
        for i in {0, 1, H // 2, H - 2, H - 1} | set(range(6, min(H, 18))):
            for j in {0, 1, W // 2, W - 2, W - 1} | set(range(6, min(W, 18))):
                if 0 <= i < H and 0 <= j < W:
                    pts.add((b * H + i) * W + j)
    rnd = rng.integers(0, B * H * W, size=n)
    return np.unique(np.concatenate([np.fromiter(pts, dtype=np.int64), rnd]))


FULL = ["c2", "c3", "c3_k5", "c3_k7", "c4", "c4_ragged", "c5", "c5_k5", "c5_k7", "c5_k9", "c5_f32"]


@pytest.mark.parametrize("name", FULL)
def test_full_size_configs_every_element(name):
    """Every output element of every full-size configuration against the oracle (the largest,
    c3_k7, is about 10 s of oracle time on 16 cores), through AUTO: what the benchmark runs."""
    cfg, x = synth.make_config(name)
    k, dtype = cfg["ksize"], cfg["dtype"]
    ref = ref_forward(x, k)
    got = gpu_forward(x, k, dtype)
    assert_close(got, ref, dtype, name)
    assert np.array_equal(got, gpu_forward(x, k, dtype)), name      # bit-identical repeat


@pytest.mark.parametrize("name", ["c2", "c5"])
def test_full_size_all_variants_agree_on_samples(name):
    cfg, x = synth.make_config(name, batch_limit=4)
    k, dtype = cfg["ksize"], cfg["dtype"]
    Bn, H, W = x["q"].shape[:3]
    pix = sample_pixels(Bn, H, W, 500, 5)
    ref = oracle.forward_pixels(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, pix)
    C = cfg["heads"] * cfg["head_dim"]
    for variant in ALL_VARIANTS:
        got = run_variant(x, k, dtype, variant)
        if got is not None:
            assert_close(got.reshape(-1, C)[pix], ref, dtype, f"{name} {variant}")


# ---- behaviour of the boundary -------------------------------------------------------------

@pytest.mark.parametrize("variant", ALL_VARIANTS)
def test_deterministic_and_leaves_guard_bands_alone(variant):
    """Two runs give identical bits; memory just before and after `out` is untouched."""
    cfg = dict(B=2, H=19, W=23, heads=3, head_dim=32, ksize=3)
    x = synth.make_inputs(**cfg, dtype="bf16", sigma_w=0.05, has_bias=True, seed=99)
    dev = to_device(x, "bf16")
    n = dev["q"].numel()
    guard = 4096
    buf = torch.full((n + 2 * guard,), -7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[guard:guard + n].view(dev["q"].shape)
    ctx = sa.slide_attn_create(cfg["B"], cfg["H"], cfg["W"], cfg["heads"], cfg["head_dim"],
                               cfg["ksize"], torch.bfloat16, True)
    try:
        if variant != "auto":
            try:
                sa.slide_attn_set_variant(ctx, VARIANTS[variant])
            except sa.SlideAttnError:
                pytest.skip("variant unsupported")
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
        first = out.clone()
        out.fill_(float("nan"))
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
        torch.cuda.synchronize()
        assert torch.equal(first.view(torch.int16), out.view(torch.int16))
        assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + n:] == -7.0).all())
        assert sa.slide_attn_query_status(ctx) == sa.OK
    finally:
        sa.slide_attn_destroy(ctx)


PIPE_SHAPES = [(64, 56, 56, 3), (7, 56, 56, 2), (33, 28, 28, 6), (5, 28, 42, 6), (2, 128, 128, 3),
               (1, 4, 8, 1), (9, 12, 72, 1), (130, 8, 8, 2), (3, 61, 67, 5)]


@pytest.mark.parametrize("shape", PIPE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_pipelined_variants_many_shapes_repeatable(shape):
    """The persistent kernels hand work between warps through mbarrier rings; shapes with many or
    few tiles per CTA, partial last blocks and ragged widths must all give the oracle's result,
    every element within the bf16 tolerance, and the same bits on every repetition."""
    B, H, W, heads = shape
    x = synth.make_inputs(B, H, W, heads, 32, 3, "bf16", 0.05, 0.1, True, seed=B * 1000 + W)
    ref = ref_forward(x, 3)
    dev = to_device(x, "bf16")
    ctx = sa.slide_attn_create(B, H, W, heads, 32, 3, torch.bfloat16, True)
    try:
        for variant in PIPELINED:
            sa.slide_attn_set_variant(ctx, VARIANTS[variant])
            outs = []
            for _ in range(4):
                o = torch.full_like(dev["q"], float("nan"))
                sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], o)
                outs.append(o)
            torch.cuda.synchronize()
            assert sa.slide_attn_query_status(ctx) == sa.OK, (variant, shape)
            for o in outs[1:]:
                assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16)), (variant, shape)
            assert_close(outs[0].float().cpu().numpy().astype(np.float64), ref, "bf16", f"{variant} {shape}")
    finally:
        sa.slide_attn_destroy(ctx)


def test_forward_argument_errors():
    x = synth.make_inputs(1, 4, 4, 1, 32, 3, "f32", seed=1, has_bias=True)
    dev = to_device(x, "f32")
    out = torch.empty_like(dev["q"])
    ctx = sa.slide_attn_create(1, 4, 4, 1, 32, 3, torch.float32, True)
    try:
        lib = sa.binding.load()
        p = lambda t: None if t is None else t.data_ptr()
        args = [p(dev[n]) for n in ("q", "k", "v", "wk", "wv", "bias")] + [p(out), None]
        assert lib.slide_attn_forward(ctx, *args) == sa.OK
        bad = list(args); bad[5] = None                      # bias missing
        assert lib.slide_attn_forward(ctx, *bad) == sa.ERR_INVALID_ARG
        bad = list(args); bad[0] = None
        assert lib.slide_attn_forward(ctx, *bad) == sa.ERR_INVALID_ARG
        bad = list(args); bad[6] = args[0]                   # out aliases q
        assert lib.slide_attn_forward(ctx, *bad) == sa.ERR_INVALID_ARG
        bad = list(args); bad[1] = args[1] + 4               # misaligned k
        assert lib.slide_attn_forward(ctx, *bad) == sa.ERR_ALIGNMENT
        assert lib.slide_attn_set_variant(ctx, 10) == sa.ERR_INVALID_ARG and lib.slide_attn_set_variant(ctx, 3) == sa.ERR_INVALID_ARG
        torch.cuda.synchronize()
    finally:
        sa.slide_attn_destroy(ctx)


@pytest.mark.parametrize("B,H,W", [(2, 11, 13), (1, 9, 20), (7, 56, 56)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_buffer_entry_point(dtype, B, H, W):
    """slide_attn_forward_host (host buffers in and out) gives the device path's result; the batch
    sizes cover one slice, two small slices and four uneven slices of its copy / compute pipeline."""
    heads, d, k = 2, 32, 3
    x = synth.make_inputs(B, H, W, heads, d, k, dtype, 0.05, 0.1, True, seed=123)
    td = TORCH_DTYPE[dtype]
    host = {n: torch.from_numpy(x[n]).to(td).pin_memory() for n in ("q", "k", "v")}
    host.update({n: torch.from_numpy(x[n]).pin_memory() for n in ("wk", "wv", "bias")})
    out = torch.empty_like(host["q"]).pin_memory()
    ctx = sa.slide_attn_create(B, H, W, heads, d, k, td, True)
    try:
        for _ in range(2):      # second call reuses the staging buffers
            out.zero_()
            sa.slide_attn_forward_host(ctx, host["q"], host["k"], host["v"], host["wk"],
                                       host["wv"], host["bias"], out)
            assert_close(out.float().numpy().astype(np.float64), ref_forward(x, k), dtype, "host entry")
    finally:
        sa.slide_attn_destroy(ctx)


def test_wrong_architecture_is_refused_not_emulated():
    major, _ = torch.cuda.get_device_capability()
    if major == 10:
        pytest.skip("this is an sm_100 device")
    with pytest.raises(sa.SlideAttnError) as e:
        sa.slide_attn_create(1, 4, 4, 1, 32, 3, torch.float32, False)
    assert e.value.status == sa.ERR_ARCH


def test_auto_random_shapes_against_oracle():
    """A seeded sweep of small random shapes (odd widths, H or W below the window, more heads than
    fit one round of CTAs, partial last blocks) through what AUTO runs for bf16 / head_dim 32 /
    k = 3, element by element against the oracle, each shape twice for bit-identical repeats."""
    rng = np.random.default_rng(20304)
    fixed = [(1, 5, 9, 160), (1, 1, 1, 300), (1, 8, 64, 149)]      # more heads than the GPU has SMs
    for it in range(48 + len(fixed)):
        if it < len(fixed):
            B, H, W, heads = fixed[it]
        else:
            B, H, W, heads = (int(rng.integers(1, 4)), int(rng.integers(1, 36)), int(rng.integers(1, 140)),
                              int(rng.integers(1, 8)))
        x = synth.make_inputs(B, H, W, heads, 32, 3, "bf16", 0.05, 0.2, bool(it & 1), seed=7000 + it)
        ref = oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], 3)
        got = gpu_forward(x, 3, "bf16")
        again = gpu_forward(x, 3, "bf16")
        assert np.array_equal(got, again), (B, H, W, heads)
        assert_close(got, ref, "bf16", f"random shape {(B, H, W, heads)}")
