"""Pins for the oracle's backward pass with the dense large kernel (ESC Section 3.2: LK of 13x13x16x16, every output
channel sums over every attention input channel; depth-wise dynamic kernel, one-layer estimator).

The dense forward is a polynomial of degree two in x and linear in each weight tensor, so differences of the PINNED
forward oracle (forward_dense) are exact up to rounding:
P42  directional derivatives in x (central differences) along random directions
P43  the same for the dense LK, W_dyn and b_dyn (one-sided differences are already exact)
P44  the diagonal case: a dense kernel that is zero off the diagonal is the depth-wise form, so gx, g_W_dyn, g_b_dyn
     must equal the PINNED depth-wise backward and the diagonal of g_w_dense its g_LK; the off-diagonal gradients are
     not zero (they are the cross-channel correlations) and are checked against a library correlation
P45  identity channels: gx = grad_out there, and they influence nothing else
A planted mistake (input and output channel swapped in g_w_dense, and in the kernel on the way back to x) breaks P42/P43.
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth

NAMES = ("x", "w_dense", "w_dyn", "b_dyn")


def _case(B=2, C=6, C_a=3, H=6, W=8, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed, channel_means=True)   # bf16 values: x +- v is exact in fp32
    d["w_dense"] = synth.make_dense_kernel(C_a, K, synth.BF16, seed=seed).astype(np.float64)
    rng = np.random.default_rng(seed + 17)
    d["go"] = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    return d, rng


def _loss(oracle, d, C_a=3, **over):
    a = {k: over.get(k, d[k]) for k in NAMES}
    out = oracle.forward_dense(a["x"], C_a, a["w_dense"], a["w_dyn"], a["b_dyn"])
    return float(np.sum(out * d["go"].astype(np.float64)))


def _grads(oracle, d, C_a=3):
    return dict(zip(NAMES, oracle.backward_dense(d["x"], d["go"], C_a, d["w_dense"], d["w_dyn"], d["b_dyn"])))


@pytest.mark.parametrize("K", [5, 3, 13])
def test_p42_directional_derivatives_in_x(oracle, K):
    d, rng = _case(K=K, H=7 if K < 13 else 15, W=9 if K < 13 else 14, seed=K)
    g = _grads(oracle, d)
    for _ in range(3):
        v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
        lp, lm = _loss(oracle, d, x=d["x"] + v), _loss(oracle, d, x=d["x"] - v)
        assert float(np.sum(g["x"] * v)) == pytest.approx((lp - lm) / 2.0, rel=1e-10, abs=1e-9)


def test_p43_weight_gradients(oracle):
    d, rng = _case(seed=43)
    g = _grads(oracle, d)
    base = _loss(oracle, d)
    for name in NAMES[1:]:
        for _ in range(3):
            v = rng.standard_normal(size=d[name].shape)
            assert float(np.sum(g[name] * v)) == pytest.approx(_loss(oracle, d, **{name: d[name].astype(np.float64) + v}) - base,
                                                               rel=1e-10, abs=1e-9), name


def test_p44_diagonal_kernel_is_the_depthwise_backward(oracle):
    import torch

    d, rng = _case(seed=44)
    C_a, K = 3, 5
    wl = d["w_large"].astype(np.float64)
    d["w_dense"] = np.zeros((C_a, C_a, K, K))
    for c in range(C_a):
        d["w_dense"][c, c] = wl[c]
    g = _grads(oracle, d)
    gx, glk, gw, gb = oracle.backward(d["x"], d["go"], C_a, wl, d["w_dyn"], d["b_dyn"])
    np.testing.assert_allclose(g["x"], gx, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["w_dyn"], gw, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["b_dyn"], gb, rtol=1e-12, atol=1e-12)
    for c in range(C_a):
        np.testing.assert_allclose(g["w_dense"][c, c], glk[c], rtol=1e-12, atol=1e-12)
    # every (n, k) block against a library correlation: g[n,k] = corr(x_k padded, go_n) summed over images
    xt = torch.from_numpy(d["x"][:, :C_a].astype(np.float64))
    gt = torch.from_numpy(d["go"][:, :C_a].astype(np.float64))
    P = (K - 1) // 2
    # conv2d with the images as channels: input [k, B, H, W], weight [n, B, H, W]  ->  [k, n, K, K]
    lib = torch.nn.functional.conv2d(xt.permute(1, 0, 2, 3), gt.permute(1, 0, 2, 3), padding=P).permute(1, 0, 2, 3).numpy()
    np.testing.assert_allclose(g["w_dense"], lib, rtol=1e-11, atol=1e-11)
    assert np.abs(g["w_dense"][0, 1]).max() > 1e-3


def test_p45_identity_channels(oracle):
    d, rng = _case(seed=45)
    C_a = 3
    g = _grads(oracle, d)
    assert np.array_equal(g["x"][:, C_a:], d["go"][:, C_a:].astype(np.float64))
    d2 = dict(d); d2["x"] = d["x"].copy(); d2["go"] = d["go"].copy()
    d2["x"][:, C_a:] += 3.0; d2["go"][:, C_a:] *= -2.0
    g2 = _grads(oracle, d2)
    assert np.array_equal(g2["x"][:, :C_a], g["x"][:, :C_a])
    for name in NAMES[1:]:
        assert np.array_equal(g2[name], g[name]), name


def test_planted_channel_swap_is_caught(oracle):
    d, rng = _case(seed=46)
    g = _grads(oracle, d)
    v = rng.standard_normal(size=d["w_dense"].shape)
    num = _loss(oracle, d, w_dense=d["w_dense"] + v) - _loss(oracle, d)
    assert float(np.sum(g["w_dense"] * v)) == pytest.approx(num, rel=1e-10, abs=1e-9)
    assert abs(float(np.sum(g["w_dense"].transpose(1, 0, 2, 3) * v)) - num) > 1e-3 * abs(num)
    # the same swap on the way back to x: the gradient of the forward with the swapped kernel
    u = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
    numx = (_loss(oracle, d, x=d["x"] + u) - _loss(oracle, d, x=d["x"] - u)) / 2.0
    wrong = oracle.backward_dense(d["x"], d["go"], 3, d["w_dense"].transpose(1, 0, 2, 3).copy(), d["w_dyn"], d["b_dyn"])[0]
    assert float(np.sum(g["x"] * u)) == pytest.approx(numx, rel=1e-10, abs=1e-9)
    assert abs(float(np.sum(wrong * u)) - numx) > 1e-3 * abs(numx)


def test_points_equal_the_pinned_whole_gradient(oracle):
    """backward_dense_points (used where the whole gradient takes too long) must return the entries of the pinned
    backward_dense, every one of them, and magnitudes that bound them."""
    d, rng = _case(B=2, C=5, C_a=3, H=7, W=9, K=5, seed=52)
    g = _grads(oracle, d)
    n = g["w_dense"].size
    vals, mags = oracle.backward_dense_points(d["x"], d["go"], 3, 5, np.arange(n))
    np.testing.assert_allclose(vals, g["w_dense"].reshape(-1), rtol=1e-13, atol=1e-13)
    assert (mags >= np.abs(vals) - 1e-12).all()

