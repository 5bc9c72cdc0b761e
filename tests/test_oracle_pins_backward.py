"""Pins for the oracle's backward pass (gradients of the ConvAttn forward of ESC Section 3.3, Eq. 4, with the
one-layer estimator and the depth-wise LK).

The forward is a polynomial of degree two in x (dk is linear in x, the output bilinear in (kernel, x)) and
linear in each weight tensor, so central differences of the PINNED forward oracle are exact up to rounding:
P24  directional derivatives in x along random directions: <gx, v> = (L(x + e v) - L(x - e v)) / (2 e)
P25  the same for LK, W_dyn and b_dyn (where a one-sided difference is already exact)
P26  identity channels: gx = grad_out there; attention gradients do not depend on them
P27  with the estimator switched off (W_dyn = 0) gx is the adjoint of a fixed linear map: <gx, v> = <grad_out, f(v) - f(0)>
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth


def _case(B=2, C=7, C_a=3, H=6, W=8, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed, channel_means=True)   # bf16 values: x +- v below is exact in fp32
    rng = np.random.default_rng(seed + 7)
    d["go"] = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    return d, rng


def _loss(oracle, d, x=None, wl=None, wd=None, bd=None, C_a=3):
    out = oracle.forward(d["x"] if x is None else x, C_a, d["w_large"] if wl is None else wl,
                         d["w_dyn"] if wd is None else wd, d["b_dyn"] if bd is None else bd)
    return float(np.sum(out * d["go"].astype(np.float64)))


@pytest.mark.parametrize("K", [5, 3, 13])
def test_p24_directional_derivatives_in_x(oracle, K):
    d, rng = _case(K=K, H=7 if K < 13 else 15, W=9 if K < 13 else 14, seed=K)
    gx, _, _, _ = oracle.backward(d["x"], d["go"], 3, d["w_large"], d["w_dyn"], d["b_dyn"])
    for _ in range(4):
        v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)      # small integers: x +- v stays exact in fp32
        lp, lm = _loss(oracle, d, x=d["x"] + v), _loss(oracle, d, x=d["x"] - v)
        assert float(np.sum(gx * v)) == pytest.approx((lp - lm) / 2.0, rel=1e-10, abs=1e-9)


def test_p25_weight_gradients(oracle):
    d, rng = _case(seed=25)
    C_a = 3
    _, glk, gw, gb = oracle.backward(d["x"], d["go"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    base = _loss(oracle, d)
    for name, g in (("w_large", glk), ("w_dyn", gw), ("b_dyn", gb)):
        for _ in range(3):
            v = rng.standard_normal(size=d[name].shape)
            kw = {"wl": None, "wd": None, "bd": None}
            kw[{"w_large": "wl", "w_dyn": "wd", "b_dyn": "bd"}[name]] = d[name].astype(np.float64) + v
            assert float(np.sum(g * v)) == pytest.approx(_loss(oracle, d, **kw) - base, rel=1e-10, abs=1e-9), name


def test_p26_identity_channels(oracle):
    d, rng = _case(seed=26)
    C_a = 3
    gx, glk, gw, gb = oracle.backward(d["x"], d["go"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    assert np.array_equal(gx[:, C_a:], d["go"][:, C_a:].astype(np.float64))
    x2, go2 = d["x"].copy(), d["go"].copy()
    x2[:, C_a:] += 3.0; go2[:, C_a:] *= -2.0
    gx2, glk2, gw2, gb2 = oracle.backward(x2, go2, C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    assert np.array_equal(gx2[:, :C_a], gx[:, :C_a]) and np.array_equal(glk2, glk) and np.array_equal(gw2, gw) and np.array_equal(gb2, gb)


def test_p27_adjoint_of_the_frozen_map(oracle):
    d, rng = _case(seed=27)
    C_a = 3
    wd0 = np.zeros_like(d["w_dyn"])
    gx, _, _, _ = oracle.backward(d["x"], d["go"], C_a, d["w_large"], wd0, d["b_dyn"])
    f0 = oracle.forward(np.zeros_like(d["x"]), C_a, d["w_large"], wd0, d["b_dyn"])
    v = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    fv = oracle.forward(v, C_a, d["w_large"], wd0, d["b_dyn"])
    assert float(np.sum(gx * v)) == pytest.approx(float(np.sum(d["go"].astype(np.float64) * (fv - f0))), rel=1e-11, abs=1e-10)
