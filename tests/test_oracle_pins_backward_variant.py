"""Pins for the oracle's backward pass of every large-kernel form with the two-layer estimator (the configurations the
paper's models use: dense LK or decomposed LK with Conv_up(GELU(Conv_down(GAP))), Section 3.2 / Eq. 4 line 2 / Eq. 5).
The oracle composes it from the pinned one-layer backward passes (generator frozen per image) and the estimator's
chain rule.

P46  the depth-wise form must equal the PINNED two-layer backward (convattn_ref_backward_mlp) to rounding: all six
     gradients
P47  dense and decomposed forms: central differences of the forward composed from pinned pieces (GAP -> dynkernel_mlp ->
     stencil_dense / stencil_pw), directional, in x and in every weight tensor; the forward is smooth, not polynomial,
     so the steps are small and the tolerance covers the O(e^2) term (as for P33)
P48  a planted mistake in a copy of the result (the estimator's path added with the wrong sign) fails P47
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth

KEYS = ("w_down", "b_down", "w_up", "b_up")


def _case(form, B=2, C=6, C_a=3, H=6, W=8, K=5, h=4, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, synth.BF16, seed=seed)
    for k in KEYS:
        d[k] = m[k].astype(np.float64)
    rng = np.random.default_rng(seed + 19)
    d["b_down"] = d["b_down"] + rng.uniform(-1.0, 1.0, size=d["b_down"].shape)      # pre-activations where phi is curved
    d["go"] = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    d["w_large"] = d["w_large"].astype(np.float64)
    d["w_point"] = synth.make_pointwise(C_a, synth.BF16, seed=seed).astype(np.float64) if form == "pw" else None
    if form == "dense":
        d["w_large"] = synth.make_dense_kernel(C_a, K, synth.BF16, seed=seed).astype(np.float64)
    return d, rng


def _forward(oracle, form, a, C_a):
    dk = oracle.dynkernel_mlp(oracle.gap(a["x"], C_a), a["w_down"], a["b_down"], a["w_up"], a["b_up"])
    if form == "dense":
        return oracle.stencil_dense(a["x"], C_a, a["w_large"], dk)
    if form == "pw":
        return oracle.stencil_pw(a["x"], C_a, a["w_large"], a["w_point"], dk)
    return oracle.stencil(a["x"], C_a, a["w_large"], dk)


def _loss(oracle, form, d, C_a=3, **over):
    a = {k: over.get(k, d[k]) for k in ("x", "w_large", "w_point") + KEYS}
    return float(np.sum(_forward(oracle, form, a, C_a) * d["go"].astype(np.float64)))


def _grads(oracle, form, d, C_a=3):
    r = oracle.backward_variant(d["x"], d["go"], C_a, form, d["w_large"], d["w_point"], *(d[k] for k in KEYS))
    return dict(zip(("x", "w_large", "w_point") + KEYS, r))


def test_p46_depthwise_form_is_the_pinned_two_layer_backward(oracle):
    d, _ = _case("depthwise", seed=46)
    g = _grads(oracle, "depthwise", d)
    ref = oracle.backward_mlp(d["x"], d["go"], 3, d["w_large"], *(d[k] for k in KEYS))
    for name, r in zip(("x", "w_large") + KEYS, ref):
        np.testing.assert_allclose(g[name], r, rtol=1e-11, atol=1e-11, err_msg=name)


@pytest.mark.parametrize("form", ["dense", "pw"])
def test_p47_central_differences(oracle, form):
    d, rng = _case(form, seed=47)
    g = _grads(oracle, form, d)
    e = 2.0 ** -12                                       # exact in fp32 on bf16-valued inputs; the O(e^2) term stays below the tolerance
    for _ in range(3):
        v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
        num = (_loss(oracle, form, d, x=d["x"] + np.float32(e) * v) - _loss(oracle, form, d, x=d["x"] - np.float32(e) * v)) / (2 * e)
        assert float(np.sum(g["x"] * v)) == pytest.approx(num, rel=1e-7, abs=5e-9 * float(np.sum(np.abs(g["x"] * v))))
    names = ("w_large",) + KEYS + (("w_point",) if form == "pw" else ())
    for name in names:
        for _ in range(2):
            v = rng.standard_normal(size=d[name].shape)
            ew = 2.0 ** -12
            num = (_loss(oracle, form, d, **{name: d[name] + ew * v}) - _loss(oracle, form, d, **{name: d[name] - ew * v})) / (2 * ew)
            assert float(np.sum(g[name] * v)) == pytest.approx(num, rel=2e-6, abs=2e-8 * float(np.sum(np.abs(g[name] * v)))), name


def test_p48_planted_sign_of_the_estimator_path(oracle):
    d, rng = _case("dense", seed=48)
    g = _grads(oracle, "dense", d)
    C_a = 3
    # the estimator's path is the part of gx that is constant per (image, channel): flip its sign in a copy
    dk = oracle.dynkernel_mlp(oracle.gap(d["x"], C_a), *(d[k] for k in KEYS)).reshape(d["x"].shape[0], -1)
    frozen = np.stack([oracle.backward_dense(d["x"][b:b + 1], d["go"][b:b + 1], C_a, d["w_large"], np.zeros((9 * C_a, C_a)), dk[b])[0][0]
                       for b in range(d["x"].shape[0])])
    const = g["x"] - frozen
    assert np.abs(const[:, :C_a]).max() > 1e-6 and np.abs(const[:, C_a:]).max() == 0.0
    wrong = frozen - const
    e = 2.0 ** -12
    v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
    num = (_loss(oracle, "dense", d, x=d["x"] + np.float32(e) * v) - _loss(oracle, "dense", d, x=d["x"] - np.float32(e) * v)) / (2 * e)
    assert float(np.sum(g["x"] * v)) == pytest.approx(num, rel=1e-7, abs=5e-9 * float(np.sum(np.abs(g["x"] * v))))
    assert abs(float(np.sum(wrong * v)) - num) > 1e-4 * abs(num)
