"""Pins for the oracle's backward pass with the estimator as the paper writes it (ESC Section 3.3, Eq. 4 line 2: two
layers with the exact GELU between them; depth-wise LK).

P33  central differences of the PINNED forward oracle (forward_mlp), directional, in x and in each of the five weight
     tensors.  The forward is smooth but no longer a polynomial (the GELU), so the differences carry an O(e^2) term;
     the steps are chosen so that it stays below the tolerance, and a wrong derivative of the GELU (the tanh form's, a
     dropped density term, a wrong sign) is shown to miss it.
P34  the linear limit: with every pre-activation shifted far to the right phi is the identity and phi' = 1, so the
     gradients must be those of the PINNED one-layer backward with the composed weights W = W_up W_down,
     b = W_up b_down + b_up:  gx and g_LK equal, g_b_up = g_b, g_W_up = g_W W_down^T + g_b b_down^T,
     g_W_down = W_up^T g_W, g_b_down = W_up^T g_b.
P35  far to the left phi = 0 and phi' = 0: nothing reaches the first layer or x through the estimator (g_W_down = 0,
     g_b_down = 0, gx = the adjoint of the fixed stencil), while the second layer's bias still gets g_dk.
P36  identity channels: gx = grad_out there, and they influence nothing else.
"""
import math

import numpy as np
import pytest

from paper_2503_06671_b200 import synth

KEYS = ("w_down", "b_down", "w_up", "b_up")


def _case(B=2, C=7, C_a=3, H=6, W=8, K=5, h=4, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed, channel_means=True)   # bf16 values: x +- e v below is exact in fp32
    m = synth.make_estimator_mlp(C_a, h, synth.BF16, seed=seed)
    for k in KEYS:
        d[k] = m[k].astype(np.float64)
    rng = np.random.default_rng(seed + 11)
    d["go"] = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    return d, rng


def _loss(oracle, d, C_a=3, **over):
    a = {k: over.get(k, d[k]) for k in ("x", "w_large") + KEYS}
    out = oracle.forward_mlp(a["x"], C_a, a["w_large"], a["w_down"], a["b_down"], a["w_up"], a["b_up"])
    return float(np.sum(out * d["go"].astype(np.float64)))


def _grads(oracle, d, C_a=3):
    g = oracle.backward_mlp(d["x"], d["go"], C_a, d["w_large"], *(d[k] for k in KEYS))
    return dict(zip(("x", "w_large") + KEYS, g))


@pytest.mark.parametrize("K,h", [(5, 4), (3, 8), (13, 5)])
def test_p33_central_differences(oracle, K, h):
    d, rng = _case(K=K, h=h, H=7 if K < 13 else 15, W=9 if K < 13 else 14, seed=K + h)
    d["b_down"] = d["b_down"] + rng.uniform(-1.0, 1.0, size=d["b_down"].shape)        # pre-activations where phi is curved
    g = _grads(oracle, d)
    # x: steps of 2^-10 on bf16-valued inputs are exact in fp32; the O(e^2) term enters through the pooled mean only
    for _ in range(3):
        v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
        e = 2.0 ** -10
        num = (_loss(oracle, d, x=d["x"] + np.float32(e) * v) - _loss(oracle, d, x=d["x"] - np.float32(e) * v)) / (2 * e)
        assert float(np.sum(g["x"] * v)) == pytest.approx(num, rel=1e-7, abs=5e-9 * float(np.sum(np.abs(g["x"] * v))))   # of the terms' scale: the sum cancels
    d["w_large"] = d["w_large"].astype(np.float64)
    for name in ("w_large",) + KEYS:
        for _ in range(2):
            v = rng.standard_normal(size=d[name].shape)
            e = 1e-5
            num = (_loss(oracle, d, **{name: d[name] + e * v}) - _loss(oracle, d, **{name: d[name] - e * v})) / (2 * e)
            assert float(np.sum(g[name] * v)) == pytest.approx(num, rel=2e-7, abs=1e-8), name


def test_p33_a_wrong_gelu_derivative_would_fail(oracle):
    """The chain through the activation, taken apart: g_W_down = (g_a * phi'(t)) g^T.  With the exact phi' the central
    difference of the pinned forward agrees; the tanh approximation's derivative and phi' without its density term
    are farther from it than the tolerance of P33."""
    d, rng = _case(seed=91, h=6)
    d["b_down"] = d["b_down"] + rng.uniform(-1.5, 1.5, size=d["b_down"].shape)
    g = _grads(oracle, d)
    C_a = 3
    gmean = oracle.gap(d["x"], C_a)
    t = gmean @ d["w_down"].T + d["b_down"]                                            # [B, h]
    gdk = oracle.backward_mlp(d["x"], d["go"], C_a, d["w_large"], *(d[k] for k in KEYS))[5]   # g_b_up = sum_b g_dk: B = 1 below
    d1, _ = _case(B=1, seed=91, h=6)
    d1["b_down"] = d["b_down"]
    g1 = _grads(oracle, d1)
    t1 = oracle.gap(d1["x"], C_a) @ d1["w_down"].T + d1["b_down"]
    ga = g1["b_up"] @ d1["w_up"]                                                       # [h]: sum_o W_up[o,m] g_dk[o]
    exact = np.array([0.5 * math.erfc(-x / math.sqrt(2)) + x * math.exp(-x * x / 2) / math.sqrt(2 * math.pi) for x in t1[0]])
    assert g1["b_down"] == pytest.approx(ga * exact, rel=1e-12, abs=1e-14)
    no_density = np.array([0.5 * math.erfc(-x / math.sqrt(2)) for x in t1[0]])
    u = math.sqrt(2 / math.pi)
    tanh_form = np.array([0.5 * (1 + math.tanh(u * (x + 0.044715 * x ** 3)))
                          + 0.5 * x * (1 - math.tanh(u * (x + 0.044715 * x ** 3)) ** 2) * u * (1 + 3 * 0.044715 * x * x) for x in t1[0]])
    assert np.abs(ga * no_density - g1["b_down"]).max() > 1e-3 * np.abs(g1["b_down"]).max()
    assert np.abs(ga * tanh_form - g1["b_down"]).max() > 1e-5 * np.abs(g1["b_down"]).max()
    # and the exact one is what the forward's central difference sees
    v = rng.standard_normal(size=d1["b_down"].shape)
    e = 1e-5
    num = (_loss(oracle, d1, b_down=d1["b_down"] + e * v) - _loss(oracle, d1, b_down=d1["b_down"] - e * v)) / (2 * e)
    assert float(np.sum(g1["b_down"] * v)) == pytest.approx(num, rel=2e-7, abs=1e-9)
    assert gdk.shape == (9 * C_a,) and t.shape == (2, 6)


@pytest.mark.parametrize("h", [4, 8, 24])
def test_p34_linear_limit_is_the_one_layer_backward(oracle, h):
    d, _ = _case(seed=34 + h, h=h, K=5)
    C_a = 3
    d["b_down"] = d["b_down"] + 40.0                   # t >= 30: Phi(t) = 1 and t n(t) = 0 in double precision
    g = _grads(oracle, d)
    Wc = d["w_up"] @ d["w_down"]
    bc = d["w_up"] @ d["b_down"] + d["b_up"]
    gx1, glk1, gw1, gb1 = oracle.backward(d["x"], d["go"], C_a, d["w_large"], Wc, bc)
    assert g["x"] == pytest.approx(gx1, rel=1e-11, abs=1e-11)
    assert g["w_large"] == pytest.approx(glk1, rel=1e-12, abs=1e-12)
    assert g["b_up"] == pytest.approx(gb1, rel=1e-12, abs=1e-12)
    assert g["w_up"] == pytest.approx(gw1 @ d["w_down"].T + np.outer(gb1, d["b_down"]), rel=1e-11, abs=1e-10)
    assert g["w_down"] == pytest.approx(d["w_up"].T @ gw1, rel=1e-11, abs=1e-11)
    assert g["b_down"] == pytest.approx(d["w_up"].T @ gb1, rel=1e-11, abs=1e-11)
    # the transposed readings differ
    assert not np.allclose(g["w_down"], (gw1.T @ d["w_up"]).T[:, ::-1], rtol=1e-6)


def test_p35_far_left_nothing_passes_the_activation(oracle):
    d, _ = _case(seed=35, h=5)
    C_a = 3
    d["b_down"] = d["b_down"] - 60.0
    g = _grads(oracle, d)
    assert np.abs(g["w_down"]).max() == 0.0 and np.abs(g["b_down"]).max() == 0.0
    assert np.abs(g["w_up"]).max() < 1e-300 or np.abs(g["w_up"]).max() == 0.0          # a = phi(t) = 0
    # dk = b_up for every image: the one-layer backward with W = 0, b = b_up gives the same gx, g_LK and g_b
    gx1, glk1, _, gb1 = oracle.backward(d["x"], d["go"], C_a, d["w_large"], np.zeros((9 * C_a, C_a)), d["b_up"])
    assert g["x"] == pytest.approx(gx1, rel=1e-12, abs=1e-12)
    assert g["w_large"] == pytest.approx(glk1, rel=1e-12, abs=1e-12)
    assert g["b_up"] == pytest.approx(gb1, rel=1e-12, abs=1e-12)


def test_p36_identity_channels(oracle):
    d, _ = _case(seed=36)
    C_a = 3
    g = _grads(oracle, d)
    assert np.array_equal(g["x"][:, C_a:], d["go"][:, C_a:].astype(np.float64))
    d2 = dict(d)
    d2["x"], d2["go"] = d["x"].copy(), d["go"].copy()
    d2["x"][:, C_a:] += 3.0
    d2["go"][:, C_a:] *= -2.0
    g2 = _grads(oracle, d2)
    assert np.array_equal(g2["x"][:, :C_a], g["x"][:, :C_a])
    for k in ("w_large",) + KEYS:
        assert np.array_equal(g2[k], g[k]), k
