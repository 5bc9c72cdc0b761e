"""Pins for the oracle's closing step of the module (ESC paper, Section 3.3, Eq. 4 line 4: F_fuse =
Conv_fuse(Concat(F_res, F_idt)), a 1x1 convolution; with the block's residual of Eq. 3 line 3).

P28  the identity matrix without bias and residual reproduces the pinned forward bit for bit
P29  a permutation matrix permutes the channels of the pinned forward exactly; a transposed reading of w_fuse fails
P30  library route: torch fp64 1x1 conv2d with bias, plus the residual
P31  pure-Python brute force per pixel; bias and residual enter once each, with weight one
P32  linearity in w_fuse, b_fuse and the residual; the returned magnitude is the sum of absolute terms
"""
import numpy as np

from paper_2503_06671_b200 import synth


def _case(B=2, C=12, C_a=4, H=9, W=11, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.F32, seed, channel_means=True)
    rng = np.random.default_rng(seed + 400)
    d["w_fuse"] = rng.uniform(-1, 1, size=(C, C))
    d["b_fuse"] = rng.uniform(-1, 1, size=(C,))
    d["res"] = rng.normal(size=(B, C, H, W)).astype(np.float32)
    return d


def test_p28_identity_matrix_is_the_forward(oracle):
    d = _case()
    cat = oracle.forward(d["x"], 4, d["w_large"], d["w_dyn"], d["b_dyn"])
    out = oracle.forward_fused(d["x"], 4, d["w_large"], d["w_dyn"], d["b_dyn"], np.eye(12))
    assert np.array_equal(out, cat)


def test_p29_permutation_matrix_and_orientation(oracle):
    d = _case(seed=1)
    C = 12
    perm = np.random.default_rng(2).permutation(C)
    P = np.zeros((C, C))
    P[np.arange(C), perm] = 1.0                     # out[n] = cat[perm[n]]
    cat = oracle.forward(d["x"], 4, d["w_large"], d["w_dyn"], d["b_dyn"])
    out = oracle.fuse(cat, P)
    assert np.array_equal(out, cat[:, perm])
    assert not np.array_equal(oracle.fuse(cat, P.T), cat[:, perm])      # rows are output channels, not columns


def test_p30_library_pointwise_convolution(oracle):
    import torch
    import torch.nn.functional as F

    d = _case(B=2, C=20, C_a=8, H=13, W=17, K=13, seed=3)
    cat = oracle.forward(d["x"], 8, d["w_large"], d["w_dyn"], d["b_dyn"])
    out = oracle.fuse(cat, d["w_fuse"], d["b_fuse"], d["res"])
    lib = F.conv2d(torch.from_numpy(cat), torch.from_numpy(d["w_fuse"])[:, :, None, None], torch.from_numpy(d["b_fuse"])).numpy()
    lib = lib + d["res"].astype(np.float64)
    assert np.abs(out - lib).max() <= 1e-12 * np.abs(lib).max()


def test_p31_brute_force_per_pixel(oracle):
    d = _case(B=1, C=6, C_a=2, H=4, W=5, K=3, seed=4)
    cat = oracle.forward(d["x"], 2, d["w_large"], d["w_dyn"], d["b_dyn"])
    out = oracle.fuse(cat, d["w_fuse"], d["b_fuse"], d["res"])
    for n in range(6):
        for y in range(4):
            for x in range(5):
                s = float(d["b_fuse"][n]) + float(d["res"][0, n, y, x])
                for c in range(6):
                    s += float(d["w_fuse"][n, c]) * float(cat[0, c, y, x])
                assert abs(out[0, n, y, x] - s) <= 1e-12 * max(1.0, abs(s))
    # bias and residual enter once, with weight one
    base = oracle.fuse(cat, d["w_fuse"])
    assert np.abs(oracle.fuse(cat, d["w_fuse"], d["b_fuse"]) - base - d["b_fuse"][None, :, None, None]).max() <= 1e-13
    assert np.abs(oracle.fuse(cat, d["w_fuse"], None, d["res"]) - base - d["res"]).max() <= 1e-13


def test_p32_linearity_and_magnitude(oracle):
    d = _case(seed=5)
    cat = oracle.forward(d["x"], 4, d["w_large"], d["w_dyn"], d["b_dyn"])
    w2 = np.random.default_rng(6).uniform(-1, 1, size=(12, 12))
    a = oracle.fuse(cat, d["w_fuse"]) * 2.0 + oracle.fuse(cat, w2) * -3.0
    b = oracle.fuse(cat, 2.0 * d["w_fuse"] - 3.0 * w2)
    assert np.abs(a - b).max() <= 1e-12 * np.abs(a).max()
    out, mag = oracle.fuse(cat, d["w_fuse"], d["b_fuse"], d["res"], want_mag=True)
    want = np.abs(d["b_fuse"])[None, :, None, None] + np.einsum("nc,bchw->bnhw", np.abs(d["w_fuse"]), np.abs(cat)) + np.abs(d["res"])
    assert np.abs(mag - want).max() <= 1e-12 * want.max()
    assert (np.abs(out) <= mag * (1 + 1e-12)).all()
