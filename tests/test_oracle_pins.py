"""Pins for the CPU oracle: it is checked against what the paper and the
mathematics fix -- the shift identity of Eq. 11-13, the column-view (Im2Col)
definition of Eq. 4-7, the re-parameterisation of Sec. 4.3, closed forms,
invariants, and library routines the method reduces to.  CPU only."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2304_04237_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_inputs(B, H, W, heads, d, k, seed, sigma_w=0.1, bias=True):
    return synth.make_inputs(B, H, W, heads, d, k, "f32", sigma_w, 0.3, bias, seed)


def run(x, k, **kw):
    return oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, **kw)


def shift_map(f, u, v):
    """g[i,j] = f[i+u, j+v], zero outside; f [B,H,W,...]."""
    B, H, W = f.shape[:3]
    g = np.zeros_like(f)
    for i in range(H):
        for j in range(W):
            if 0 <= i + u < H and 0 <= j + v < W:
                g[:, i, j] = f[:, i + u, j + v]
    return g


# ---- step 1: shift as depthwise convolution (Eq. 10-13) -------------------

def test_topleft_one_hot_kernel_reads_up_left_neighbour():
    """The paper's own example: k=3, kernel with the 1 at top-left gives
    f[i-1, j-1] (Eq. 10-13).  Slot 0 of the fixed-shift weights is that kernel."""
    f = np.arange(1, 1 + 2 * 4 * 5 * 3, dtype=np.float32).reshape(2, 4, 5, 3)
    w = synth.one_hot_weights(3, 3)
    assert w[0, 0].reshape(3, 3)[0, 0] == 1.0 and w[0, 0].sum() == 1.0
    y = oracle.dwconv(f, w, 3)
    want = shift_map(f, -1, -1)
    assert np.array_equal(y[:, :, :, 0, :], want.astype(np.float64))
    assert y[0, 0, 0, 0, 0] == 0.0 and y[0, 1, 1, 0, 0] == f[0, 0, 0, 0]


@pytest.mark.parametrize("k", [1, 3, 5, 7])
def test_every_one_hot_slot_is_a_shift_bit_exact(k):
    """Row view (Eq. 8-9): slot (u,v) of the fixed kernels is the map shifted by
    (u,v), zero where it leaves the map; integer maps, exact equality."""
    rng = np.random.default_rng(k)
    f = rng.integers(-50, 50, size=(2, 5, 6, 4)).astype(np.float32)
    y = oracle.dwconv(f, synth.one_hot_weights(4, k), k)
    r = k // 2
    for u in range(-r, r + 1):
        for v in range(-r, r + 1):
            s = (u + r) * k + (v + r)
            assert np.array_equal(y[:, :, :, s, :], shift_map(f, u, v).astype(np.float64)), (u, v)


@pytest.mark.parametrize("k", [3, 5])
def test_dwconv_matches_library_group_convolution(k):
    """Sec. 4.2: the k*k depthwise convolutions are one group convolution with
    C*k*k output channels and groups=C -- a library routine (conv2d is a
    cross-correlation, like Eq. 12).  Output channel index is c*k*k + slot."""
    C, k2 = 6, k * k
    f = synth.normal(11, 0, 2 * 7 * 9 * C).reshape(2, 7, 9, C).astype(np.float32)
    w = synth.normal(11, 1, C * k2 * k2).reshape(C, k2, k2).astype(np.float32)
    y = oracle.dwconv(f, w, k)
    ft = torch.from_numpy(f).double().permute(0, 3, 1, 2)
    wt = torch.from_numpy(w).double().reshape(C * k2, 1, k, k)
    yt = F.conv2d(ft, wt, padding=k // 2, groups=C)           # [B, C*k2, H, W]
    yt = yt.reshape(2, C, k2, 7, 9).permute(0, 3, 4, 2, 1).numpy()
    assert np.abs(y - yt).max() < 1e-12


# ---- whole path against the column view (Eq. 4-7) and the two-path form ----

@pytest.mark.parametrize("H,W,k", [(2, 2, 3), (1, 1, 3), (3, 5, 3), (5, 3, 5), (1, 4, 5),
                                   (7, 7, 3), (2, 3, 1), (4, 4, 7)])
def test_matches_im2col_brute_force_on_tiny_maps(H, W, k):
    """With the fixed-shift kernels the convolution form must give exactly what
    explicit window gathering gives (end of Sec. 4.1); 2x2 with k=3 is the
    example of Fig. 2."""
    x = rand_inputs(2, H, W, 2, 4, k, seed=100 + H * 10 + W + k)
    C = 8
    E = synth.one_hot_weights(C, k)
    got = oracle.forward(x["q"], x["k"], x["v"], E, E, x["bias"], k)
    want = oracle.im2col_local_attention(x["q"], x["k"], x["v"], k, x["bias"])
    assert np.abs(got - want).max() < 1e-12


@pytest.mark.parametrize("k", [3, 5])
def test_two_path_equals_merged(k):
    """Re-parameterisation (Sec. 4.3 (3), Fig. 4): shift path + learned path
    equals one convolution with the summed kernel."""
    x = rand_inputs(1, 4, 5, 2, 4, k, seed=7 + k)
    C = 8
    E = synth.one_hot_weights(C, k)
    Dk, Dv = x["wk"] - E, x["wv"] - E
    got = run(x, k)
    want = oracle.two_path_forward(x["q"], x["k"], x["v"], E, Dk, Dv, k, x["bias"])
    assert np.abs(got - want).max() < 1e-6     # wk = fl32(E + D): 1e-6 covers that rounding
    # and exactly, when the merged kernel is formed without rounding (D on a coarse grid)
    Dk = np.round(Dk * 64) / 64
    Dv = np.round(Dv * 64) / 64
    got = oracle.forward(x["q"], x["k"], x["v"], E + Dk, E + Dv, x["bias"], k)
    want = oracle.two_path_forward(x["q"], x["k"], x["v"], E, Dk, Dv, k, x["bias"])
    assert np.abs(got - want).max() < 1e-12


@pytest.mark.parametrize("k,heads,d", [(3, 2, 4), (5, 1, 8), (3, 3, 2)])
def test_matches_library_composition(k, heads, d):
    """conv2d(groups=C) -> per-head dot with q -> softmax -> weighted sum, all
    library ops in float64: the unfused pipeline of Sec. 4.  Random dense
    weights catch a transposed slot/tap index; bias catches the head/slot order."""
    B, H, W = 2, 6, 5
    C, k2 = heads * d, k * k
    x = rand_inputs(B, H, W, heads, d, k, seed=31 * k + heads, sigma_w=0.7)
    got = run(x, k)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).double()
    def expand(f, w):
        y = F.conv2d(t(f).reshape(B, H, W, C).permute(0, 3, 1, 2), t(w).reshape(C * k2, 1, k, k),
                     padding=k // 2, groups=C)
        return y.reshape(B, heads, d, k2, H, W).permute(0, 4, 5, 1, 3, 2)   # [B,H,W,heads,k2,d]
    Ks, Vs = expand(x["k"], x["wk"]), expand(x["v"], x["wv"])
    l = torch.einsum("bijhd,bijhsd->bijhs", t(x["q"]), Ks) / d ** 0.5 + t(x["bias"])
    a = torch.softmax(l, dim=-1)
    want = torch.einsum("bijhs,bijhsd->bijhd", a, Vs).numpy()
    assert np.abs(got - want).max() < 1e-11


# ---- closed forms -----------------------------------------------------------

def test_k1_is_pointwise_scaling_of_v():
    """k=1: one slot, softmax == 1, so out = wv[c] * v whatever q, k, bias are."""
    x = rand_inputs(2, 3, 4, 2, 4, 1, seed=5)
    got = run(x, 1)
    want = x["v"].astype(np.float64) * x["wv"].astype(np.float64).reshape(2, 4)
    assert np.abs(got - want).max() < 1e-15
    x["wv"] = np.ones_like(x["wv"])
    assert np.array_equal(run(x, 1), x["v"].astype(np.float64))


def test_single_pixel_map_closed_form():
    """H=W=1, k=3, fixed kernels: only the centre slot is inside the map.  Padded
    slots have key 0, hence logit 0, and keep their share of the softmax:
    out = v * e^l / (e^l + 8), l = q.k / sqrt(d).  Pins the 1/sqrt(d) scale and
    the treatment of padding (zero keys/values, not masked)."""
    d = 16
    q = np.full((1, 1, 1, 1, d), 0.5, np.float32)
    k = np.full((1, 1, 1, 1, d), 0.75, np.float32)
    v = np.arange(d, dtype=np.float32).reshape(1, 1, 1, 1, d)
    E = synth.one_hot_weights(d, 3)
    got = oracle.forward(q, k, v, E, E, None, 3)
    l = d * 0.5 * 0.75 / 4.0            # sqrt(16) = 4
    want = v * (np.exp(l) / (np.exp(l) + 8.0))
    assert np.abs(got - want).max() < 1e-13
    assert abs(l - 1.5) < 1e-15


def test_zero_query_gives_padded_box_filter_of_v():
    """q = 0, no bias: all logits 0, uniform attention 1/k^2, so with the fixed
    kernels out is the mean of the zero-padded window = average pooling with
    padded cells counted (a library routine)."""
    k = 3
    x = rand_inputs(2, 6, 7, 2, 4, k, seed=9, bias=False)
    x["q"][:] = 0
    E = synth.one_hot_weights(8, k)
    got = oracle.forward(x["q"], x["k"], x["v"], E, E, None, k)
    vt = torch.from_numpy(x["v"]).double().reshape(2, 6, 7, 8).permute(0, 3, 1, 2)
    want = F.avg_pool2d(vt, k, stride=1, padding=1, count_include_pad=True)
    want = want.permute(0, 2, 3, 1).reshape(2, 6, 7, 2, 4).numpy()
    assert np.abs(got - want).max() < 1e-14


def test_uniform_keys_with_deformed_values_is_mean_of_value_slots():
    """Uniform attention with deformed V kernels: out = (1/k^2) * conv(v; sum over
    slots of the kernels) -- one ordinary depthwise convolution."""
    k, C = 3, 8
    x = rand_inputs(1, 5, 6, 2, 4, k, seed=10, bias=False, sigma_w=0.5)
    x["k"][:] = 0
    got = run(x, k)
    wsum = torch.from_numpy(x["wv"]).double().sum(1).reshape(C, 1, k, k)
    vt = torch.from_numpy(x["v"]).double().reshape(1, 5, 6, C).permute(0, 3, 1, 2)
    want = (F.conv2d(vt, wsum, padding=1, groups=C) / 9.0).permute(0, 2, 3, 1).reshape(got.shape).numpy()
    assert np.abs(got - want).max() < 1e-13


def test_constant_values_interior_one_border_partial():
    """v = 1 with fixed kernels: every in-map slot has value 1, padded ones 0.
    Interior out = 1 (softmax rows sum to 1); with q = 0 a border pixel gets
    (#in-map slots)/k^2."""
    k = 3
    x = rand_inputs(1, 5, 5, 1, 4, k, seed=12, bias=False)
    x["v"][:] = 1
    E = synth.one_hot_weights(4, k)
    got = oracle.forward(x["q"], x["k"], x["v"], E, E, None, k)
    assert np.abs(got[:, 1:-1, 1:-1] - 1.0).max() < 1e-15
    x["q"][:] = 0
    got = oracle.forward(x["q"], x["k"], x["v"], E, E, None, k)
    assert np.abs(got[0, 0, 0] - 4.0 / 9.0).max() < 1e-15      # corner: 4 of 9 slots inside
    assert np.abs(got[0, 0, 2] - 6.0 / 9.0).max() < 1e-15      # edge: 6 of 9


@pytest.mark.parametrize("k", [3, 5])
def test_saturating_bias_selects_one_slot_exactly(k):
    """bias = 0 on one slot and -1000 elsewhere, q = 0: attention is exactly
    one-hot, so out is v shifted by that slot's offset.  Pins the bias
    [heads, slot] order and the slot -> offset map through the whole path."""
    heads, d, r, k2 = 2, 2, k // 2, k * k
    rng = np.random.default_rng(3)
    v = rng.integers(0, 200, size=(1, 6, 7, heads, d)).astype(np.float32)
    q = np.zeros_like(v)
    kk = rng.standard_normal(v.shape).astype(np.float32)
    E = synth.one_hot_weights(heads * d, k)
    slots = [(0, k2 - 1), (1, k2 // 2), (k, 2)]        # (slot for head 0, slot for head 1)
    for s0, s1 in slots:
        bias = np.full((heads, k2), -1000.0, np.float32)
        bias[0, s0] = 0
        bias[1, s1] = 0
        got = oracle.forward(q, kk, v, E, E, bias, k)
        for h, s in ((0, s0), (1, s1)):
            u, vv = s // k - r, s % k - r
            assert np.array_equal(got[:, :, :, h], shift_map(v, u, vv)[:, :, :, h].astype(np.float64))


# ---- invariants -------------------------------------------------------------

def test_attention_rows_sum_to_one_and_ignore_logit_offset():
    k = 3
    x = rand_inputs(2, 5, 4, 2, 4, k, seed=21)
    out, attn = run(x, k, return_attn=True)
    assert np.abs(attn.sum(-1) - 1.0).max() < 1e-15
    assert attn.min() > 0
    x2 = dict(x)
    x2["bias"] = x["bias"] + np.array([[3.0], [-2.0]], np.float32)   # constant per head
    out2 = run(x2, k)
    assert np.abs(out - out2).max() < 1e-6      # fp32 bias + offset rounds at ~1e-7


def test_translation_equivariance_on_interior_pixels():
    """Shifting q, k, v by (dy, dx) shifts the output, on pixels whose windows
    stay inside the map in both runs (Sec. 3.2 (3))."""
    k, r, dy, dx = 3, 1, 2, 1
    H, W = 9, 8
    x = rand_inputs(1, H, W, 2, 4, k, seed=33)
    out = run(x, k)
    y = dict(x)
    for n in ("q", "k", "v"):
        y[n] = np.roll(x[n], (dy, dx), axis=(1, 2))
    out_s = run(y, k)
    a = out[:, r:H - r - dy, r:W - r - dx]
    b = out_s[:, r + dy:H - r, r + dx:W - r]
    assert a.size > 0 and np.array_equal(a, b)


def test_heads_are_independent_and_order_is_head_major():
    """Changing head 1's q must not change head 0's output (channel c = h*d + e)."""
    k = 3
    x = rand_inputs(1, 4, 4, 2, 4, k, seed=41)
    out = run(x, k)
    x["q"][:, :, :, 1] *= -2
    out2 = run(x, k)
    assert np.array_equal(out[:, :, :, 0], out2[:, :, :, 0])
    assert np.abs(out[:, :, :, 1] - out2[:, :, :, 1]).max() > 1e-3


def test_pixel_sampler_matches_full_forward():
    k = 3
    x = rand_inputs(2, 5, 6, 2, 4, k, seed=51)
    out = run(x, k).reshape(-1, 8)
    pix = np.array([0, 7, 29, 30, 59], dtype=np.int64)
    got = oracle.forward_pixels(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, pix)
    assert np.array_equal(got, out[pix])


def test_rejects_even_window():
    """Even k has no centred window (u, v range over [-floor(k/2), floor(k/2)])."""
    x = rand_inputs(1, 3, 3, 1, 4, 3, seed=1)
    w = np.zeros((4, 4, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.forward(x["q"], x["k"], x["v"], w, w, None, 2)


# ---- stored values (written by tests/golden/make_golden.py from the oracle) --

def test_golden_samples_of_tiny_config():
    """Guards the oracle against silent change: sampled outputs of the tiny
    configuration, stored as text."""
    path = os.path.join(GOLDEN, "c1_tiny_samples.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    cfg, x = synth.make_config("c1_tiny")
    out = run(x, cfg["ksize"]).reshape(-1)
    for idx, val in rows:
        assert abs(out[int(idx)] - float(val)) <= 1e-12 * max(1.0, abs(float(val)))
