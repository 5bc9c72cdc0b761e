"""Pins for the oracle's two-layer kernel estimator (ESC paper, Section 3.3, Eq. 4 line 2:
DK = Conv_up(phi(Conv_down(GAP(F_att)))), phi the Gaussian error linear unit t * Phi(t)).

P9   phi against tabulated values of the standard normal distribution function Phi and against an
     independent implementation of Phi (scipy.special.ndtr) on a grid
P10  reflection law phi(t) - phi(-t) = t
P11  the two linear limits: pre-activations far right of zero make phi the identity, so the estimator
     collapses to the one-layer estimator with composed weights (already pinned); far left, to b_up
P12  pure-Python brute force with math.erf for the paper's hidden widths 4, 8 and 24
P13  whole forward in the linear limit equals the pinned one-layer forward with composed weights
"""
import math

import numpy as np
import pytest
from scipy import special

from paper_2503_06671_b200 import synth

# Phi(t) from a table of the standard normal distribution (values to 16 digits).
PHI_TABLE = {
    0.0: 0.5,
    0.5: 0.6914624612740131,
    1.0: 0.8413447460685429,
    2.0: 0.9772498680518208,
    3.0: 0.9986501019683699,
    -1.0: 0.15865525393145707,
    -2.0: 0.022750131948179195,
}


def _phi_through_oracle(oracle, t):
    """phi(t) read out of the estimator: one channel, one hidden unit, unit weights, g = t."""
    g = np.array([[t]], dtype=np.float64)
    w_up = np.zeros((9, 1)); w_up[0, 0] = 1.0
    dk, hid = oracle.dynkernel_mlp(g, np.ones((1, 1)), np.zeros(1), w_up, np.zeros(9), want_hidden=True)
    assert dk.reshape(9)[0] == hid[0, 0] and not dk.reshape(9)[1:].any()
    return hid[0, 0]


@pytest.mark.parametrize("t", sorted(PHI_TABLE))
def test_p9_gelu_tabulated(oracle, t):
    got = _phi_through_oracle(oracle, t)
    assert got == pytest.approx(t * PHI_TABLE[t], rel=1e-14, abs=1e-16)
    # the tanh approximation of the same unit is a different function: this pin tells them apart
    if t != 0.0:
        approx = 0.5 * t * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (t + 0.044715 * t ** 3)))
        assert abs(approx - t * PHI_TABLE[t]) > 1e-5 * abs(t)


def test_p9b_gelu_grid_against_independent_phi(oracle):
    ts = np.linspace(-8.0, 8.0, 321)
    got = np.array([_phi_through_oracle(oracle, float(t)) for t in ts])
    want = ts * special.ndtr(ts)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-300)
    assert got[ts < 0].max() <= 0.0 and (got[ts > 0] > 0.0).all()


def test_p10_reflection_law(oracle):
    rng = np.random.default_rng(10)
    C_a = 6
    g = rng.uniform(-4, 4, size=(3, C_a))
    w_up = np.zeros((9 * C_a, C_a))
    for c in range(C_a):
        w_up[c * 9 + 4, c] = 1.0          # hidden unit c -> centre tap of channel c
    args = (np.eye(C_a), np.zeros(C_a), w_up, np.zeros(9 * C_a))
    dp = oracle.dynkernel_mlp(g, *args)
    dm = oracle.dynkernel_mlp(-g, *args)
    assert np.allclose((dp - dm)[:, :, 1, 1], g, rtol=1e-14, atol=1e-15)
    others = np.ones((3, 3), bool); others[1, 1] = False
    assert not dp[:, :, others].any()


@pytest.mark.parametrize("h", [4, 8, 24])
def test_p11_linear_limits(oracle, h):
    C_a = 16
    rng = np.random.default_rng(h)
    g = rng.uniform(-2, 2, size=(5, C_a))
    m = synth.make_estimator_mlp(C_a, h, synth.F32, seed=3)
    wd, wu, bu = (m[k].astype(np.float64) for k in ("w_down", "w_up", "b_up"))
    shift = 40.0                                           # |W_down g| <= 16 * 1 * 2 = 32 < 40
    bd = m["b_down"].astype(np.float64) * 0.1 + shift
    dk = oracle.dynkernel_mlp(g, wd, bd, wu, bu)
    lin = oracle.dynkernel(g, wu @ wd, wu @ bd + bu)       # one-layer estimator, composed weights
    assert np.allclose(dk, lin, rtol=1e-12, atol=1e-12)
    dk0 = oracle.dynkernel_mlp(g, wd, bd - 2 * shift, wu, bu)
    assert np.allclose(dk0.reshape(5, -1), np.broadcast_to(bu, (5, 9 * C_a)), rtol=0, atol=1e-300)


@pytest.mark.parametrize("h", [4, 8, 24])
def test_p12_brute_force(oracle, h):
    C_a, B = 3, 2
    rng = np.random.default_rng(100 + h)
    g = rng.uniform(-1.5, 1.5, size=(B, C_a))
    wd = rng.uniform(-1, 1, size=(h, C_a)); bd = rng.uniform(-1, 1, size=h)
    wu = rng.uniform(-1, 1, size=(9 * C_a, h)); bu = rng.uniform(-1, 1, size=9 * C_a)
    dk, hid = oracle.dynkernel_mlp(g, wd, bd, wu, bu, want_hidden=True)
    for b in range(B):
        a = []
        for j in range(h):
            t = math.fsum([bd[j]] + [wd[j, c] * g[b, c] for c in range(C_a)])
            a.append(t * 0.5 * (1.0 + math.erf(t / math.sqrt(2.0))))     # t * Phi(t), Phi written with erf
            assert hid[b, j] == pytest.approx(a[j], rel=1e-13, abs=1e-15)
        for c in range(C_a):
            for i in range(3):
                for jj in range(3):
                    o = c * 9 + i * 3 + jj
                    want = math.fsum([bu[o]] + [wu[o, j] * a[j] for j in range(h)])
                    assert dk[b, c, i, jj] == pytest.approx(want, rel=1e-12, abs=1e-14)


def test_p13_forward_linear_limit_is_pinned_forward(oracle):
    B, C, C_a, H, W, K, h = 2, 10, 4, 9, 11, 5, 8
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.F32, seed=13, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, synth.F32, seed=13)
    wd, wu, bu = (m[k].astype(np.float64) for k in ("w_down", "w_up", "b_up"))
    bd = np.full(h, 60.0)
    out, dk = oracle.forward_mlp(d["x"], C_a, d["w_large"], wd, bd, wu, bu, want_dk=True)
    ref, dk_ref = oracle.forward(d["x"], C_a, d["w_large"], wu @ wd, wu @ bd + bu, want_dk=True)
    assert np.allclose(dk, dk_ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(out, ref, rtol=1e-11, atol=1e-11)
    assert np.array_equal(out[:, C_a:], d["x"][:, C_a:].astype(np.float64))
    # and away from the limit the activation matters: the same weights with b_down = 0 give another dk
    dk_mid = oracle.dynkernel_mlp(oracle.gap(d["x"], C_a), wd, np.zeros(h), wu, bu)
    assert np.abs(dk_mid - oracle.dynkernel(oracle.gap(d["x"], C_a), wu @ wd, bu)).max() > 1e-2
