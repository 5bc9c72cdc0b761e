"""Pins for the CPU oracle: checks against what the definition (ESC paper, Section 3.3,
Eq. 4 and Eq. 5) and plain mathematics fix, none of which re-type the oracle's own loops.

P0  hand-evaluated 2x2 example (tests/golden/hand_2x2_k3.txt)
P1  impulse input reproduces the 180-degree-rotated summed kernels
P2  constant input gives the border-truncated kernel sums (summed-area closed form)
P3  zero generator reduces to a library depth-wise convolution (torch fp64 conv2d)
P4  scatter-form brute force on tiny inputs (incl. H,W < K, 1xW, Hx1)
P5  linearity laws (frozen dk linear; quadratic scaling law; zero-mean perturbation)
P6  Eq. 5 merge identity ZP(DK)+LK
P7  channel permutation, batch independence, identity channels never leak
P8  GAP -> dk stage on non-zero-mean data against math.fsum
"""
import math
import os

import numpy as np
import pytest

from paper_2503_06671_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(B, C, C_a, H, W, K=13, seed=0, **kw):
    return synth.make_inputs(B, C, C_a, H, W, K, synth.F32, seed, **kw)


def test_p0_hand_example(oracle):
    rows = [l for l in open(os.path.join(GOLDEN, "hand_2x2_k3.txt")) if not l.startswith("#")]
    expect = np.array([[float(v) for v in r.split()] for r in rows]).reshape(1, 2, 2, 2)
    x = np.array([[[[1, 2], [3, 4]], [[5, 6], [7, 8]]]], dtype=np.float32)
    w_large = np.array([[[1, 0, -1], [2, 0, -2], [1, 0, -1]]], dtype=np.float64)
    w_dyn = np.zeros((9, 1)); w_dyn[4, 0] = 2.0
    b_dyn = np.zeros(9); b_dyn[1] = 1.0
    out, dk = oracle.forward(x, 1, w_large, w_dyn, b_dyn, want_dk=True)
    assert np.array_equal(dk.reshape(3, 3), np.array([[0, 1, 0], [0, 5, 0], [0, 0, 0]], dtype=float))
    assert np.array_equal(out, expect)


@pytest.mark.parametrize("pos", [(20, 17), (0, 0), (2, 30), (31, 4), (5, 5), (31, 31)])
def test_p1_impulse(oracle, pos):
    B, C, C_a, H, W, K, P = 1, 6, 4, 32, 32, 13, 6
    d = _rand(B, C, C_a, H, W, K, seed=11)
    c0, (y0, x0) = 2, pos
    x = np.zeros((B, C, H, W), dtype=np.float32)
    x[0, c0, y0, x0] = 1.0
    out, dk = oracle.forward(x, C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_dk=True)
    # dk from the definition: g = delta/HW in channel c0 only
    dk_expect = (d["w_dyn"][:, c0].astype(np.float64) / (H * W) + d["b_dyn"]).reshape(C_a, 3, 3)
    np.testing.assert_allclose(dk[0], dk_expect, rtol=1e-14, atol=0)
    expect = np.zeros((H, W))
    for di in range(-P, P + 1):
        for dj in range(-P, P + 1):
            y, xx = y0 - di, x0 - dj
            if 0 <= y < H and 0 <= xx < W:
                v = float(d["w_large"][c0, di + P, dj + P])
                if abs(di) <= 1 and abs(dj) <= 1:
                    v += dk_expect[c0, di + 1, dj + 1]
                expect[y, xx] = v
    np.testing.assert_allclose(out[0, c0], expect, rtol=1e-14, atol=0)
    for c in range(C_a):
        if c != c0:
            assert not out[0, c].any()           # other attention channels: exactly zero
    assert not out[0, C_a:].any()                # identity channels copy the zeros


def _truncated_box_sums(w, H, W):
    """S(y,x) = sum of the taps of w that fall inside an HxW image when centred at (y,x)."""
    K = w.shape[-1]
    P = (K - 1) // 2
    sat = np.zeros((K + 1, K + 1))
    sat[1:, 1:] = np.cumsum(np.cumsum(w.astype(np.float64), 0), 1)
    S = np.empty((H, W))
    for y in range(H):
        i0, i1 = max(0, P - y), min(K - 1, P + H - 1 - y)
        for x in range(W):
            j0, j1 = max(0, P - x), min(K - 1, P + W - 1 - x)
            S[y, x] = sat[i1 + 1, j1 + 1] - sat[i0, j1 + 1] - sat[i1 + 1, j0] + sat[i0, j0]
    return S


@pytest.mark.parametrize("H,W", [(20, 24), (7, 9), (13, 40)])
def test_p2_constant_closed_form(oracle, H, W):
    B, C, C_a, K = 2, 5, 3, 13
    d = _rand(B, C, C_a, H, W, K, seed=5)
    alpha = np.array([[0.5, -1.25, 2.0, 3.0, -0.75], [1.5, 0.25, -2.0, 1.0, 4.0]], dtype=np.float32)
    x = np.broadcast_to(alpha[:, :, None, None], (B, C, H, W)).copy()
    out, dk = oracle.forward(x, C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_dk=True)
    for b in range(B):
        a = alpha[b, :C_a].astype(np.float64)
        dk_expect = (d["w_dyn"].astype(np.float64) @ a + d["b_dyn"]).reshape(C_a, 3, 3)
        np.testing.assert_allclose(dk[b], dk_expect, rtol=1e-13, atol=1e-15)
        for c in range(C_a):
            S = _truncated_box_sums(d["w_large"][c], H, W) + _truncated_box_sums(dk_expect[c], H, W)
            np.testing.assert_allclose(out[b, c], a[c] * S, rtol=1e-11, atol=1e-12)
        for c in range(C_a, C):
            assert np.array_equal(out[b, c], x[b, c].astype(np.float64))


@pytest.mark.parametrize("K", [13, 9, 3])
def test_p3_zero_generator_is_library_depthwise_conv(oracle, K):
    torch = pytest.importorskip("torch")
    B, C, C_a, H, W = 2, 8, 4, 23, 31
    d = _rand(B, C, C_a, H, W, K, seed=7)
    out = oracle.forward(d["x"], C_a, d["w_large"], np.zeros_like(d["w_dyn"]), np.zeros_like(d["b_dyn"]))
    xt = torch.from_numpy(d["x"][:, :C_a].astype(np.float64))
    wt = torch.from_numpy(d["w_large"].astype(np.float64)).unsqueeze(1)
    ref = torch.nn.functional.conv2d(xt, wt, padding=(K - 1) // 2, groups=C_a).numpy()
    np.testing.assert_allclose(out[:, :C_a], ref, rtol=1e-12, atol=1e-12)
    assert np.array_equal(out[:, C_a:], d["x"][:, C_a:].astype(np.float64))


def test_p3b_full_op_is_two_library_convs(oracle):
    """With the generator on: out = conv(x, LK) + per-image conv(x, dk), dk from a separate mean."""
    torch = pytest.importorskip("torch")
    B, C, C_a, H, W, K = 3, 6, 4, 19, 22, 13
    d = _rand(B, C, C_a, H, W, K, seed=8, channel_means=True)
    out = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    xt = torch.from_numpy(d["x"][:, :C_a].astype(np.float64))
    lk = torch.nn.functional.conv2d(xt, torch.from_numpy(d["w_large"].astype(np.float64)).unsqueeze(1),
                                    padding=6, groups=C_a)
    g = xt.mean(dim=(2, 3))
    dk = g @ torch.from_numpy(d["w_dyn"].astype(np.float64)).T + torch.from_numpy(d["b_dyn"].astype(np.float64))
    for b in range(B):
        dyn = torch.nn.functional.conv2d(xt[b:b + 1], dk[b].reshape(C_a, 1, 3, 3), padding=1, groups=C_a)
        np.testing.assert_allclose(out[b, :C_a], (lk[b] + dyn[0]).numpy(), rtol=1e-11, atol=1e-12)


def _scatter_form(x, C_a, w_large, dk):
    """Second implementation: loop over INPUT pixels and scatter each into the outputs it touches."""
    B, C, H, W = x.shape
    K = w_large.shape[-1]
    out = np.zeros((B, C, H, W))
    for b in range(B):
        for c in range(C_a):
            for ys in range(H):
                for xs in range(W):
                    v = float(x[b, c, ys, xs])
                    for w, k in ((w_large[c], K), (dk[b, c], 3)):
                        p = (k - 1) // 2
                        for i in range(k):
                            for j in range(k):
                                y, xx = ys - i + p, xs - j + p
                                if 0 <= y < H and 0 <= xx < W:
                                    out[b, c, y, xx] += float(w[i, j]) * v
        out[b, C_a:] = x[b, C_a:]
    return out


@pytest.mark.parametrize("H,W", [(5, 5), (1, 17), (15, 1), (13, 13), (14, 20), (2, 3)])
def test_p4_scatter_brute_force(oracle, H, W):
    B, C, C_a, K = 2, 3, 2, 13
    d = _rand(B, C, C_a, H, W, K, seed=3 + H * 31 + W, channel_means=True)
    out, dk = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_dk=True)
    g = d["x"][:, :C_a].astype(np.float64).reshape(B, C_a, -1).sum(-1) / (H * W)
    dk_ind = (g @ d["w_dyn"].astype(np.float64).T + d["b_dyn"]).reshape(B, C_a, 3, 3)
    np.testing.assert_allclose(dk, dk_ind, rtol=1e-12, atol=1e-14)
    ref = _scatter_form(d["x"], C_a, d["w_large"].astype(np.float64), dk_ind)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)


def test_p4b_5x5_every_output_sees_every_pixel(oracle):
    """K=13 > H,W: out[y,x] = sum_{y',x'} w[y'-y+6, x'-x+6] x[y',x'] (+ 3x3 term)."""
    d = _rand(1, 1, 1, 5, 5, 13, seed=21)
    z9 = np.zeros((9, 1)); zb = np.zeros(9)
    out = oracle.forward(d["x"], 1, d["w_large"], z9, zb)
    x = d["x"][0, 0].astype(np.float64); w = d["w_large"][0].astype(np.float64)
    for y in range(5):
        for xx in range(5):
            assert out[0, 0, y, xx] == pytest.approx((w[6 - y:11 - y, 6 - xx:11 - xx] * x).sum(), rel=1e-12, abs=1e-13)


def test_p5_linearity_laws(oracle):
    B, C, C_a, H, W, K = 2, 5, 4, 17, 21, 13
    d = _rand(B, C, C_a, H, W, K, seed=31, channel_means=True)
    x1 = d["x"]
    x2 = _rand(B, C, C_a, H, W, K, seed=32)["x"]
    wl, wd, bd = d["w_large"], d["w_dyn"], d["b_dyn"]
    # (i) frozen generator (W_dyn = 0): f is linear in x. Use inputs whose combination is exact in f32.
    x1q = np.round(x1 * 64) / 64; x2q = np.round(x2 * 64) / 64
    xc = (0.5 * x1q + 2.0 * x2q).astype(np.float32)
    assert np.array_equal(xc.astype(np.float64), 0.5 * x1q.astype(np.float64) + 2.0 * x2q.astype(np.float64))
    f = lambda x: oracle.forward(x, C_a, wl, np.zeros_like(wd), bd)
    # with b_dyn != 0 and W_dyn = 0 the op is linear (dk is a constant kernel)
    np.testing.assert_allclose(f(xc), 0.5 * f(x1q) + 2.0 * f(x2q), rtol=1e-12, atol=1e-12)
    # (ii) stencil stage: linear in w_large and in dk
    dk1 = np.random.default_rng(1).standard_normal((B, C_a, 3, 3))
    dk2 = np.random.default_rng(2).standard_normal((B, C_a, 3, 3))
    s = lambda w, dk: oracle.stencil(x1q, C_a, w, dk)[:, :C_a]
    w2 = _rand(B, C, C_a, H, W, K, seed=33)["w_large"].astype(np.float64)
    lhs = s(2.0 * wl.astype(np.float64) + w2, 3.0 * dk1 - dk2)
    rhs = 2.0 * s(wl, 0 * dk1) + s(w2, 0 * dk1) + 3.0 * (s(0 * w2, dk1)) - s(0 * w2, dk2)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-11, atol=1e-11)
    # (iii) quadratic scaling law with b_dyn = 0: f(s x) = s L(x) + s^2 D(x)
    z = np.zeros_like(bd)
    full = lambda x: oracle.forward(x, C_a, wl, wd, z)[:, :C_a]
    L = oracle.forward(x1q, C_a, wl, np.zeros_like(wd), z)[:, :C_a]
    D = full(x1q) - L
    for sc in (2.0, -0.5, 4.0):
        np.testing.assert_allclose(full((sc * x1q).astype(np.float32)), sc * L + sc * sc * D, rtol=1e-10, atol=1e-10)
    # ... and the full op is NOT linear (guards against a generator that ignores x)
    assert np.abs(full((2.0 * x1q).astype(np.float32)) - 2.0 * full(x1q)).max() > 1e-3
    # (iv) zero-mean perturbation leaves dk unchanged: f(x1+x2) = f(x1) + LK*x2 + DK(x1)*x2
    x2z = x2q[:, :, :, :].astype(np.float64)
    x2z = x2z - x2z.mean(axis=(2, 3), keepdims=True)
    x2z = np.round(x2z * 4096) / 4096
    x2z[:, :, 0, 0] -= x2z.sum(axis=(2, 3))        # exact zero sum (all values are multiples of 2^-12)
    assert np.abs(x2z.sum(axis=(2, 3))).max() == 0.0
    x2z32 = x2z.astype(np.float32); assert np.array_equal(x2z32.astype(np.float64), x2z)
    xsum = (x1q.astype(np.float64) + x2z).astype(np.float32)
    assert np.array_equal(xsum.astype(np.float64), x1q.astype(np.float64) + x2z)
    _, dk_x1 = oracle.forward(x1q, C_a, wl, wd, bd, want_dk=True)
    lhs = oracle.forward(xsum, C_a, wl, wd, bd)[:, :C_a]
    rhs = oracle.forward(x1q, C_a, wl, wd, bd)[:, :C_a] + oracle.stencil(x2z32, C_a, wl, dk_x1)[:, :C_a]
    np.testing.assert_allclose(lhs, rhs, rtol=1e-10, atol=1e-10)


def test_p6_merge_identity(oracle):
    """Eq. 5: one convolution with ZP(DK)+LK equals the sum of the two convolutions."""
    B, C, C_a, H, W, K, P = 2, 4, 4, 18, 16, 13, 6
    d = _rand(B, C, C_a, H, W, K, seed=41, channel_means=True)
    out, dk = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_dk=True)
    for b in range(B):
        merged = d["w_large"].astype(np.float64).copy()
        merged[:, P - 1:P + 2, P - 1:P + 2] += dk[b]
        ob = oracle.stencil(d["x"][b:b + 1], C_a, merged, np.zeros((1, C_a, 3, 3)))
        np.testing.assert_allclose(ob[0], out[b], rtol=1e-12, atol=1e-13)


def test_p7_permutation_batch_independence_no_leak(oracle):
    B, C, C_a, H, W, K = 3, 7, 4, 16, 15, 13
    d = _rand(B, C, C_a, H, W, K, seed=51, channel_means=True)
    x, wl, wd, bd = d["x"], d["w_large"], d["w_dyn"], d["b_dyn"]
    out = oracle.forward(x, C_a, wl, wd, bd)
    # permute attention channels together with the matching weights
    perm = np.array([2, 0, 3, 1])
    xp = x.copy(); xp[:, :C_a] = x[:, perm]
    rows = (perm[:, None] * 9 + np.arange(9)[None, :]).reshape(-1)
    outp = oracle.forward(xp, C_a, wl[perm], wd[rows][:, perm], bd[rows])
    np.testing.assert_allclose(outp[:, :C_a], out[:, perm], rtol=1e-12, atol=1e-13)
    # images are independent
    for b in range(B):
        ob = oracle.forward(x[b:b + 1], C_a, wl, wd, bd)
        assert np.array_equal(ob[0], out[b])
    # identity channels never influence attention channels, and pass through exactly
    x2 = x.copy(); x2[:, C_a:] = 1e6 * np.sign(x[:, C_a:])
    out2 = oracle.forward(x2, C_a, wl, wd, bd)
    assert np.array_equal(out2[:, :C_a], out[:, :C_a])
    assert np.array_equal(out2[:, C_a:], x2[:, C_a:].astype(np.float64))
    # attention channels do not mix in the stencil: changing channel 1 changes only dk-coupled terms;
    # with W_dyn = 0 there is no coupling at all
    x3 = x.copy(); x3[:, 1] += 3.0
    o_a = oracle.forward(x, C_a, wl, np.zeros_like(wd), bd)
    o_b = oracle.forward(x3, C_a, wl, np.zeros_like(wd), bd)
    keep = [0, 2, 3]
    assert np.array_equal(o_a[:, keep], o_b[:, keep])
    assert not np.array_equal(o_a[:, 1], o_b[:, 1])


def test_p8_dk_stage_nonzero_mean(oracle):
    B, C, C_a, H, W = 2, 6, 4, 33, 47
    d = _rand(B, C, C_a, H, W, 13, seed=61, channel_means=True)
    g = oracle.gap(d["x"], C_a)
    for b in range(B):
        for c in range(C_a):
            exact = math.fsum(float(v) for v in d["x"][b, c].ravel()) / (H * W)
            assert g[b, c] == pytest.approx(exact, rel=1e-13)
    dk = oracle.dynkernel(g, d["w_dyn"], d["b_dyn"])
    for b in range(B):
        for o in range(9 * C_a):
            exact = math.fsum([float(d["b_dyn"][o])] + [float(d["w_dyn"][o, c]) * g[b, c] for c in range(C_a)])
            assert dk.reshape(B, -1)[b, o] == pytest.approx(exact, rel=1e-12, abs=1e-15)
    # the generator really depends on the mean: shifting a channel by t moves dk by t * W_dyn[:, c]
    x2 = d["x"].copy(); x2[:, 2] += 2.0
    dk2 = oracle.dynkernel(oracle.gap(x2, C_a), d["w_dyn"], d["b_dyn"])
    np.testing.assert_allclose((dk2 - dk).reshape(B, -1), np.broadcast_to(2.0 * d["w_dyn"][:, 2].astype(np.float64), (B, 9 * C_a)), rtol=1e-6, atol=1e-7)


def test_rows_and_points_agree_with_forward(oracle):
    B, C, C_a, H, W = 2, 5, 3, 21, 18
    d = _rand(B, C, C_a, H, W, 13, seed=71, channel_means=True)
    out, mag, dk = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True, want_dk=True)
    band = oracle.stencil(d["x"], C_a, d["w_large"], dk, rows=(4, 13))
    assert np.array_equal(band, out[:, :, 4:13])
    idx = np.random.default_rng(0).integers(0, out.size, size=200)
    vals, mags = oracle.points(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], idx, want_mag=True)
    assert np.array_equal(vals, out.ravel()[idx])
    assert (mags >= np.abs(vals) - 1e-12).all()
    oracle.set_threads(1)
    out1 = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    oracle.set_threads(oracle.max_threads())
    assert np.array_equal(out1, out)            # thread count does not change a single bit
