"""Pins of the backward oracle (oracle/backward.py) against things other than itself: central finite
differences of the FORWARD oracle, the two-path identity of Sec. 4.3, k = 1, softmax invariants; and
the host-side re-parameterisation utility against the forward oracle's two-path form."""
import numpy as np
import pytest

import oracle
from oracle import backward as ob
from paper_2304_04237_b200 import reparam, synth


def grid(rng, shape, scale=1.0):
    """Values on a 1/64 grid: x +- 2**-9 is then exact in float, so finite differences of the float-input
    forward oracle see exactly the perturbation asked for."""
    return (np.round(rng.normal(size=shape) * scale * 64) / 64).astype(np.float32)


def problem(seed, B=1, H=4, W=5, heads=2, d=4, k=3, bias=True, dense=False):
    rng = np.random.default_rng(seed)
    C, k2 = heads * d, k * k
    x = dict(q=grid(rng, (B, H, W, heads, d)), k=grid(rng, (B, H, W, heads, d)), v=grid(rng, (B, H, W, heads, d)))
    dlt = grid(rng, (C, k2, k2), 0.3 if dense else 0.05)
    x["wk"] = (synth.one_hot_weights(C, k) + dlt).astype(np.float32)
    x["wv"] = (synth.one_hot_weights(C, k) + grid(rng, (C, k2, k2), 0.3 if dense else 0.05)).astype(np.float32)
    x["bias"] = grid(rng, (heads, k2), 0.5) if bias else None
    x["dout"] = rng.normal(size=(B, H, W, heads, d))
    return x, k


def loss(x, k):
    return float((oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k) * x["dout"]).sum())


def finite_difference(x, k, name, idx, eps=2.0 ** -9):
    hi, lo = dict(x), dict(x)
    hi[name] = x[name].copy(); lo[name] = x[name].copy()
    hi[name][idx] += eps; lo[name][idx] -= eps
    assert hi[name][idx] - lo[name][idx] == np.float32(2 * eps)       # the step is exact in float
    return (loss(hi, k) - loss(lo, k)) / (2 * eps)


@pytest.mark.parametrize("cfg", [dict(seed=1), dict(seed=2, k=5, H=5, W=4, heads=1, d=3), dict(seed=3, H=2, W=2),
                                 dict(seed=4, bias=False, dense=True), dict(seed=5, B=2, H=3, W=3, heads=3, d=2),
                                 dict(seed=6, H=1, W=1), dict(seed=7, k=1)])
def test_backward_matches_finite_differences_of_the_forward(cfg):
    x, k = problem(**cfg)
    g = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, x["dout"])
    rng = np.random.default_rng(99)
    for name, grad in (("q", g["dq"]), ("k", g["dk"]), ("v", g["dv"]), ("wk", g["dwk"]), ("wv", g["dwv"]), ("bias", g["dbias"])):
        if x[name] is None:
            assert grad is None
            continue
        assert grad.shape == x[name].shape
        picks = [tuple(rng.integers(0, n) for n in x[name].shape) for _ in range(12)]
        picks += [tuple(0 for _ in x[name].shape), tuple(n - 1 for n in x[name].shape)]      # corners: padding paths
        for idx in picks:
            fd = finite_difference(x, k, name, idx)
            assert abs(fd - grad[idx]) <= 2e-5 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


def test_every_element_against_finite_differences_on_a_tiny_problem():
    """All entries of all six gradients (a transposed slot/tap, a flipped shift or a dropped padding
    term anywhere shows up here)."""
    x, k = problem(seed=11, H=2, W=3, heads=1, d=2, k=3)
    g = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, x["dout"])
    for name, grad in (("q", g["dq"]), ("k", g["dk"]), ("v", g["dv"]), ("wk", g["dwk"]), ("wv", g["dwv"]), ("bias", g["dbias"])):
        for idx in np.ndindex(*x[name].shape):
            fd = finite_difference(x, k, name, idx)
            assert abs(fd - grad[idx]) <= 2e-5 * max(1.0, abs(fd)), (name, idx)


def test_softmax_invariants_and_k1():
    x, k = problem(seed=21)
    g = ob.backward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k, x["dout"])
    # adding a constant to all logits of a head changes nothing: the bias gradient sums to zero over slots
    assert np.abs(g["dbias"].sum(-1)).max() < 1e-12
    # k = 1: one slot, attention == 1, out = wv * v: dq = dk = 0, dv = wv * dout, dwv = sum dout * v
    x1, _ = problem(seed=22, k=1)
    g1 = ob.backward(x1["q"], x1["k"], x1["v"], x1["wk"], x1["wv"], x1["bias"], 1, x1["dout"])
    B, H, W, heads, d = x1["q"].shape
    assert np.abs(g1["dq"]).max() == 0 and np.abs(g1["dk"]).max() == 0 and np.abs(g1["dwk"]).max() == 0
    wv = x1["wv"].reshape(heads, d).astype(np.float64)
    np.testing.assert_allclose(g1["dv"], wv * x1["dout"], atol=1e-12)
    np.testing.assert_allclose(g1["dwv"].reshape(heads, d), (x1["dout"] * x1["v"]).sum((0, 1, 2)), atol=1e-12)


def test_two_path_gradients_and_the_merge_utility():
    """Sec. 4.3: merged = shift + learned.  The utility's merged kernel gives the two-path forward; the
    learned kernels' gradient is the merged kernels' gradient (finite differences through the two-path
    forward oracle)."""
    x, k = problem(seed=31, heads=1, d=3)
    C = x["wk"].shape[0]
    E = reparam.shift_kernels(C, k)
    assert np.array_equal(E, synth.one_hot_weights(C, k))
    Dk, Dv = reparam.split_merged(x["wk"], k), reparam.split_merged(x["wv"], k)
    assert np.array_equal(reparam.merge_two_path(Dk, k), x["wk"])
    torch_layout = Dv.reshape(C * k * k, 1, k, k)                    # a depthwise conv weight with groups = C
    assert np.array_equal(reparam.merge_two_path(torch_layout, k), x["wv"])
    merged = oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], k)
    two = oracle.two_path_forward(x["q"], x["k"], x["v"], E, Dk, Dv, k, x["bias"])
    np.testing.assert_allclose(merged, two, atol=1e-12)
    g = ob.two_path_backward(x["q"], x["k"], x["v"], E, Dk, Dv, x["bias"], k, x["dout"])
    eps = 2.0 ** -9
    rng = np.random.default_rng(5)
    for _ in range(10):
        idx = tuple(rng.integers(0, n) for n in Dk.shape)
        hi, lo = Dk.copy(), Dk.copy()
        hi[idx] += eps; lo[idx] -= eps
        f = lambda D: float((oracle.two_path_forward(x["q"], x["k"], x["v"], E, D, Dv, k, x["bias"]) * x["dout"]).sum())
        fd = (f(hi) - f(lo)) / (2 * eps)
        assert abs(fd - g["dlearned_wk"][idx]) <= 2e-5 * max(1.0, abs(fd))
