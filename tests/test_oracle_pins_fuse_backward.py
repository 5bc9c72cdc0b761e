"""Pins for the oracle's backward pass of Conv_fuse (ESC Eq. 4 line 4 with the block's residual, Eq. 3 line 3).

The forward is linear in its input and in each weight, so differences of the PINNED forward (fuse) are exact:
P49  <g_cat, v> = L(cat + v) - L(cat);  <g_w, u> = L(w + u) - L(w);  <g_b, t> = L(b + t) - L(b)
P50  the identity matrix: g_cat = grad_out; a permutation matrix carries grad_out's channels back through the permutation
     (row = output channel), and g_w is the channel-by-channel correlation matrix (against numpy's einsum)
P51  planted: the weight transposed on the way back, and g_w transposed, each break P49
"""
import numpy as np
import pytest


def _case(B=2, C=5, H=4, W=6, seed=0):
    rng = np.random.default_rng(seed)
    cat = (np.round(rng.standard_normal((B, C, H, W)) * 64) / 64).astype(np.float32)      # few bits: cat + v below is exact in fp32
    go = rng.standard_normal((B, C, H, W)).astype(np.float32)
    w = rng.standard_normal((C, C))
    b = rng.standard_normal((C,))
    res = rng.standard_normal((B, C, H, W)).astype(np.float32)
    return cat, go, w, b, res, rng


def _loss(oracle, cat, go, w, b, res):
    return float(np.sum(oracle.fuse(cat, w, b, res) * go.astype(np.float64)))


def test_p49_exact_differences(oracle):
    cat, go, w, b, res, rng = _case(seed=49)
    g_cat, g_w, g_b = oracle.fuse_backward(cat, go, w)
    base = _loss(oracle, cat, go, w, b, res)
    for _ in range(3):
        v = rng.integers(-2, 3, size=cat.shape).astype(np.float32)
        assert float(np.sum(g_cat * v)) == pytest.approx(_loss(oracle, cat + v, go, w, b, res) - base, rel=1e-10, abs=1e-9)
        u = rng.standard_normal(w.shape)
        assert float(np.sum(g_w * u)) == pytest.approx(_loss(oracle, cat, go, w + u, b, res) - base, rel=1e-10, abs=1e-9)
        t = rng.standard_normal(b.shape)
        assert float(np.sum(g_b * t)) == pytest.approx(_loss(oracle, cat, go, w, b + t, res) - base, rel=1e-10, abs=1e-9)


def test_p50_identity_and_permutation(oracle):
    cat, go, w, b, res, rng = _case(seed=50)
    C = cat.shape[1]
    g_cat, g_w, g_b = oracle.fuse_backward(cat, go, np.eye(C))
    assert np.array_equal(g_cat, go.astype(np.float64))
    np.testing.assert_allclose(g_w, np.einsum("bnyx,bcyx->nc", go.astype(np.float64), cat.astype(np.float64)), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g_b, go.astype(np.float64).sum(axis=(0, 2, 3)), rtol=1e-12, atol=1e-12)
    perm = np.array([3, 0, 4, 1, 2])
    Pm = np.zeros((C, C)); Pm[np.arange(C), perm] = 1.0            # out[n] = cat[perm[n]]
    g_cat, _, _ = oracle.fuse_backward(cat, go, Pm)
    want = np.empty_like(g_cat); want[:, perm] = go.astype(np.float64)
    assert np.array_equal(g_cat, want)


def test_p51_planted_transpositions(oracle):
    cat, go, w, b, res, rng = _case(seed=51)
    g_cat, g_w, _ = oracle.fuse_backward(cat, go, w)
    base = _loss(oracle, cat, go, w, b, res)
    v = rng.integers(-2, 3, size=cat.shape).astype(np.float32)
    num = _loss(oracle, cat + v, go, w, b, res) - base
    wrong_cat, _, _ = oracle.fuse_backward(cat, go, w.T.copy())
    assert abs(float(np.sum(wrong_cat * v)) - num) > 1e-3 * abs(num)
    u = rng.standard_normal(w.shape)
    numw = _loss(oracle, cat, go, w + u, b, res) - base
    assert abs(float(np.sum(g_w.T * u)) - numw) > 1e-3 * abs(numw)
