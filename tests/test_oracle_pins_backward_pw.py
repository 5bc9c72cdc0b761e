"""Pins for the oracle's backward pass of the decomposed form (ESC Eq. 5: the point-wise LK^c in front of the
depth-wise stage; one-layer estimator fed by the GAP of the unmixed features).

The decomposed forward is still a polynomial of degree two in x and linear in each weight tensor (LK^s, LK^c, W_dyn,
b_dyn), so differences of the PINNED forward oracle (forward_pw) are exact up to rounding:
P37  directional derivatives in x (central differences) along random directions
P38  the same for LK^s, LK^c, W_dyn and b_dyn (one-sided differences are already exact)
P39  the identity mix: every gradient the depth-wise form has must equal the PINNED depth-wise backward, and the
     gradient of LK^c must then be  sum_{b,pixels} gx_stencil[n] * x[k]  with gx_stencil the depth-wise backward's gx
     without its GAP constant (obtained from the pinned backward with W_dyn = 0 and b_dyn = the frozen dk)
P40  a permutation mix: mixing by a permutation matrix is the depth-wise form on permuted channels, so gx is the
     pinned backward's gx (of the permuted problem) carried back through the permutation
P41  identity channels: gx = grad_out there, and they influence nothing else
Planted mistakes (in copies of the oracle's result, on the CPU) show that P37/P38 separate the plausible errors: LK^c
transposed on the way back, the estimator's term taken from the mixed mean, a dropped GAP constant.
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth

NAMES = ("x", "w_large", "w_point", "w_dyn", "b_dyn")


def _case(B=2, C=7, C_a=3, H=6, W=8, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed, channel_means=True)   # bf16 values: x +- v is exact in fp32
    d["w_point"] = synth.make_pointwise(C_a, synth.BF16, seed=seed).astype(np.float64)
    rng = np.random.default_rng(seed + 13)
    d["go"] = rng.standard_normal(size=d["x"].shape).astype(np.float32)
    return d, rng


def _loss(oracle, d, C_a=3, **over):
    a = {k: over.get(k, d[k]) for k in NAMES}
    out = oracle.forward_pw(a["x"], C_a, a["w_large"], a["w_point"], a["w_dyn"], a["b_dyn"])
    return float(np.sum(out * d["go"].astype(np.float64)))


def _grads(oracle, d, C_a=3):
    return dict(zip(NAMES, oracle.backward_pw(d["x"], d["go"], C_a, d["w_large"], d["w_point"], d["w_dyn"], d["b_dyn"])))


@pytest.mark.parametrize("K", [5, 3, 13])
def test_p37_directional_derivatives_in_x(oracle, K):
    d, rng = _case(K=K, H=7 if K < 13 else 15, W=9 if K < 13 else 14, seed=K)
    g = _grads(oracle, d)
    for _ in range(4):
        v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
        lp, lm = _loss(oracle, d, x=d["x"] + v), _loss(oracle, d, x=d["x"] - v)
        assert float(np.sum(g["x"] * v)) == pytest.approx((lp - lm) / 2.0, rel=1e-10, abs=1e-9)


def test_p38_weight_gradients(oracle):
    d, rng = _case(seed=38)
    g = _grads(oracle, d)
    base = _loss(oracle, d)
    for name in NAMES[1:]:
        for _ in range(3):
            v = rng.standard_normal(size=d[name].shape)
            assert float(np.sum(g[name] * v)) == pytest.approx(_loss(oracle, d, **{name: d[name].astype(np.float64) + v}) - base,
                                                               rel=1e-10, abs=1e-9), name


def test_p39_identity_mix_is_the_depthwise_backward(oracle):
    d, rng = _case(seed=39)
    C_a = 3
    d["w_point"] = np.eye(C_a)
    g = _grads(oracle, d)
    gx, glk, gw, gb = oracle.backward(d["x"], d["go"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    np.testing.assert_allclose(g["x"], gx, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["w_large"], glk, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["w_dyn"], gw, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["b_dyn"], gb, rtol=1e-12, atol=1e-12)
    # dL/dm from the pinned backward with the generator frozen at this input's dk
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    gm = np.stack([oracle.backward(d["x"][b:b + 1], d["go"][b:b + 1], C_a, d["w_large"], np.zeros_like(d["w_dyn"]),
                                   dk[b].reshape(-1))[0][0, :C_a] for b in range(d["x"].shape[0])])
    want = np.einsum("bnyx,bkyx->nk", gm, d["x"][:, :C_a].astype(np.float64))
    np.testing.assert_allclose(g["w_point"], want, rtol=1e-11, atol=1e-11)


def test_p40_permutation_mix(oracle):
    d, rng = _case(C=6, C_a=4, seed=40)
    C_a = 4
    perm = np.array([2, 0, 3, 1])
    Pm = np.zeros((C_a, C_a)); Pm[np.arange(C_a), perm] = 1.0          # m[n] = x[perm[n]]
    d["w_point"] = Pm
    d["w_dyn"] = np.zeros_like(d["w_dyn"])                             # the estimator sees unpermuted means: keep it out of this pin
    g = dict(zip(NAMES, oracle.backward_pw(d["x"], d["go"], C_a, d["w_large"], Pm, d["w_dyn"], d["b_dyn"])))
    xp = d["x"].copy(); xp[:, :C_a] = d["x"][:, perm]
    gx, glk, _, gb = oracle.backward(xp, d["go"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    back = np.empty_like(gx); back[:, C_a:] = gx[:, C_a:]; back[:, perm] = gx[:, :C_a]
    np.testing.assert_allclose(g["x"], back, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["w_large"], glk, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["b_dyn"], gb, rtol=1e-12, atol=1e-12)


def test_p41_identity_channels(oracle):
    d, rng = _case(seed=41)
    C_a = 3
    g = _grads(oracle, d)
    assert np.array_equal(g["x"][:, C_a:], d["go"][:, C_a:].astype(np.float64))
    d2 = dict(d); d2["x"] = d["x"].copy(); d2["go"] = d["go"].copy()
    d2["x"][:, C_a:] += 3.0; d2["go"][:, C_a:] *= -2.0
    g2 = _grads(oracle, d2)
    assert np.array_equal(g2["x"][:, :C_a], g["x"][:, :C_a])
    for name in NAMES[1:]:
        assert np.array_equal(g2[name], g[name]), name


def test_planted_mistakes_are_caught(oracle):
    """Each plausible error, planted in a copy of the oracle's result, breaks the difference pins."""
    d, rng = _case(seed=42)
    C_a, (B, C, H, W) = 3, d["x"].shape
    g = _grads(oracle, d)
    v = rng.integers(-2, 3, size=d["x"].shape).astype(np.float32)
    num = (_loss(oracle, d, x=d["x"] + v) - _loss(oracle, d, x=d["x"] - v)) / 2.0
    assert float(np.sum(g["x"] * v)) == pytest.approx(num, rel=1e-10, abs=1e-9)
    # the GAP constant and dL/dm, separated with the frozen generator
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    frozen = np.stack([oracle.backward_pw(d["x"][b:b + 1], d["go"][b:b + 1], C_a, d["w_large"], d["w_point"],
                                          np.zeros_like(d["w_dyn"]), dk[b].reshape(-1))[0][0] for b in range(B)])
    const = g["x"][:, :C_a] - frozen[:, :C_a]                          # g_g / (H W), constant per (image, channel)
    assert np.allclose(const, const[:, :, :1, :1]) and np.abs(const).max() > 1e-6
    # (1) LK^c applied un-transposed on the way back
    gm = np.linalg.solve(d["w_point"].T, frozen[:, :C_a].transpose(1, 0, 2, 3).reshape(C_a, -1)).reshape(C_a, B, H, W).transpose(1, 0, 2, 3)
    wrong = g["x"].copy(); wrong[:, :C_a] = np.einsum("kn,bnyx->bkyx", d["w_point"], gm) + const
    assert abs(float(np.sum(wrong * v)) - num) > 1e-3 * abs(num)
    # (2) dropped GAP constant
    wrong = g["x"].copy(); wrong[:, :C_a] -= const
    assert abs(float(np.sum(wrong * v)) - num) > 1e-6 * abs(num)
    # (3) g_W formed with the mean of the mixed features
    gmean = oracle.gap(d["x"], C_a)
    wrong_gw = np.einsum("bo,bk->ok", np.stack([oracle.backward_pw(d["x"][b:b + 1], d["go"][b:b + 1], C_a, d["w_large"], d["w_point"],
                                                                   d["w_dyn"], d["b_dyn"])[4] for b in range(B)]),
                         gmean @ d["w_point"].T)
    u = rng.standard_normal(size=d["w_dyn"].shape)
    numw = _loss(oracle, d, w_dyn=d["w_dyn"].astype(np.float64) + u) - _loss(oracle, d)
    assert float(np.sum(g["w_dyn"] * u)) == pytest.approx(numw, rel=1e-10, abs=1e-9)
    assert abs(float(np.sum(wrong_gw * u)) - numw) > 1e-3 * abs(numw)
