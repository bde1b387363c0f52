"""Pins of the block oracle (oracle/block.py: Eq. 1 projections, the local attention, Eq. 3 output
projection) against things other than itself: explicit loops over Eq. 1 and Eq. 3, identity projections
(the block is then the attention stage alone), the closed form on a 1 x 1 map, a channel permutation that
moves whole heads, and the bf16 rounding helper against a library conversion."""
import numpy as np
import pytest
import torch

import oracle
from oracle import block as ob
from paper_2304_04237_b200 import synth


def problem(seed, B=1, H=3, W=4, heads=2, d=4, k=3, bias=True):
    rng = np.random.default_rng(seed)
    C, k2 = heads * d, k * k
    p = dict(x=rng.normal(size=(B, H, W, C)).astype(np.float32))
    for name in ("w_q", "w_k", "w_v", "w_o"):
        p[name] = (rng.normal(size=(C, C)) / np.sqrt(C)).astype(np.float32)
    p["wk"] = (synth.one_hot_weights(C, k) + 0.05 * rng.normal(size=(C, k2, k2))).astype(np.float32)
    p["wv"] = (synth.one_hot_weights(C, k) + 0.05 * rng.normal(size=(C, k2, k2))).astype(np.float32)
    p["bias"] = (0.3 * rng.normal(size=(heads, k2))).astype(np.float32) if bias else None
    return p, k, heads


def run(p, k, heads, **kw):
    return ob.block_forward(p["x"], p["w_q"], p["w_k"], p["w_v"], p["w_o"], p["wk"], p["wv"], p["bias"], k, heads, **kw)


def test_projection_is_eq1_written_as_loops():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(2, 3, 5))
    w = rng.normal(size=(5, 4))
    want = np.zeros((2, 3, 4))
    for a in range(2):
        for b in range(3):
            for o in range(4):
                for i in range(5):
                    want[a, b, o] += x[a, b, i] * w[i, o]          # token row times W, input channel i -> output o
    np.testing.assert_allclose(ob.project(x, w), want, rtol=0, atol=1e-13)


@pytest.mark.parametrize("cfg", [dict(seed=1), dict(seed=2, k=5, heads=1, d=6), dict(seed=3, B=2, H=2, W=2, heads=3, d=2, bias=False),
                                 dict(seed=4, k=1)])
def test_block_is_the_three_stages_in_order(cfg):
    """Eq. 1, the attention of `oracle.forward` on the projected tensors split into heads (channel = head * d +
    element), Eq. 3: the projections here are explicit loops, so a transposed weight, a swapped w_k / w_v or a
    wrong head split fails."""
    p, k, heads = problem(**cfg)
    out, q, kk, v, z = run(p, k, heads, return_parts=True)
    B, H, W, C = p["x"].shape
    d = C // heads
    x64 = p["x"].astype(np.float64)

    def loops(w):
        r = np.zeros((B, H, W, C))
        for o in range(C):
            for i in range(C):
                r[..., o] += x64[..., i] * float(w[i, o])
        return r

    for got, w in ((q, p["w_q"]), (kk, p["w_k"]), (v, p["w_v"])):
        np.testing.assert_allclose(got.reshape(B, H, W, C), loops(w), rtol=0, atol=1e-12)
    for h in range(heads):                                            # head h alone sees channels h*d .. h*d+d-1
        sl = slice(h * d, h * d + d)
        zh = oracle.forward(q[..., h:h + 1, :].astype(np.float32), kk[..., h:h + 1, :].astype(np.float32),
                            v[..., h:h + 1, :].astype(np.float32), p["wk"][sl], p["wv"][sl],
                            None if p["bias"] is None else p["bias"][h:h + 1], k)
        np.testing.assert_allclose(z[..., sl], zh.reshape(B, H, W, d), rtol=0, atol=1e-12)
    want = np.zeros((B, H, W, C))
    for o in range(C):
        for i in range(C):
            want[..., o] += z[..., i] * float(p["w_o"][i, o])
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_identity_projections_leave_the_attention_stage():
    p, k, heads = problem(5)
    C = p["x"].shape[-1]
    eye = np.eye(C, dtype=np.float32)
    for name in ("w_q", "w_k", "w_v", "w_o"):
        p[name] = eye
    B, H, W, _ = p["x"].shape
    x5 = p["x"].reshape(B, H, W, heads, C // heads)
    want = oracle.forward(x5, x5, x5, p["wk"], p["wv"], p["bias"], k).reshape(B, H, W, C)
    np.testing.assert_allclose(run(p, k, heads), want, rtol=0, atol=1e-12)


def test_one_pixel_map_closed_form():
    """H = W = 1, k = 1: one slot, softmax weight 1, so z = wv * (x W_v) and out = z W_o whatever q and k are."""
    p, _, heads = problem(6, H=1, W=1, k=1)
    xv = p["x"].astype(np.float64) @ p["w_v"].astype(np.float64)
    want = (xv * p["wv"][:, 0, 0].astype(np.float64)) @ p["w_o"].astype(np.float64)
    np.testing.assert_allclose(run(p, 1, heads), want, rtol=0, atol=1e-6)    # v passes through float on its way in


def test_swapping_heads_by_permuting_projection_columns():
    """Exchanging the column blocks of W_q, W_k, W_v that feed head 0 and head 1 (and the matching channels of
    the depthwise weights, bias rows and W_o rows) must not change the block output."""
    p, k, heads = problem(7, heads=2, d=3)
    d = 3
    perm = np.r_[np.arange(d, 2 * d), np.arange(0, d)]
    s = dict(p)
    for name in ("w_q", "w_k", "w_v"):
        s[name] = p[name][:, perm]
    s["w_o"] = p["w_o"][perm, :]
    s["wk"], s["wv"] = p["wk"][perm], p["wv"][perm]
    s["bias"] = p["bias"][[1, 0]]
    np.testing.assert_allclose(run(s, k, heads), run(p, k, heads), rtol=0, atol=1e-12)


def test_output_projection_is_linear():
    p, k, heads = problem(8)
    a = run(p, k, heads)
    p2 = dict(p); p2["w_o"] = (2.0 * p["w_o"]).astype(np.float32)
    np.testing.assert_allclose(run(p2, k, heads), 2.0 * a, rtol=0, atol=1e-12)


def test_round_bf16_matches_a_library_conversion_and_ties_go_to_even():
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.normal(size=4096), rng.normal(size=512) * 1e-3, rng.normal(size=512) * 1e4]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)
    np.testing.assert_array_equal(ob.round_bf16(x), want)
    # 1 + 2^-8 lies halfway between the bf16 neighbours 1 and 1 + 2^-7: even mantissa wins (1.0);
    # 1 + 3 * 2^-8 lies halfway between 1 + 2^-7 and 1 + 2^-6: even mantissa is 1 + 2^-6
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    np.testing.assert_array_equal(ob.round_bf16(ties), [1.0, 1.0 + 2.0 ** -6])


def test_bf16_storage_rounds_q_k_v_and_z_once_each():
    p, k, heads = problem(10)
    out, q, kk, v, z = run(p, k, heads, storage="bf16", return_parts=True)
    for t in (q, kk, v, z):
        np.testing.assert_array_equal(t, ob.round_bf16(t))
    out64, q64, _, _, _ = run(p, k, heads, storage="f64", return_parts=True)
    np.testing.assert_array_equal(q, ob.round_bf16(q64))
    assert np.abs(out - out64).max() < 0.05 and np.abs(out - out64).max() > 0
