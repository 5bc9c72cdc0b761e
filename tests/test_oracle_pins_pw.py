"""Pins for the oracle's decomposed large kernel (ESC paper, Section 3.3, Eq. 5:
F_res = (F_att * LK^c) * (ZP(DK) + LK^s), LK^c a 1x1 convolution over the 16 attention channels).

P14  identity LK^c gives back the pinned depth-wise forward, bit for bit
P15  library route: torch fp64 1x1 conv2d, then depth-wise conv2d with LK^s and with dk
P16  a spatial kernel shared by all channels commutes with the mix: out = LK^c applied per pixel to the
     pinned depth-wise result (tells LK^c from its transpose)
P17  a permutation as LK^c equals the pinned stencil on permuted channels; the output is linear in LK^c
P18  pure-Python brute force on a tiny map (borders included)
P19  dk comes from GAP of the unmixed features; identity channels pass through untouched
"""
import math

import numpy as np
import pytest

from paper_2503_06671_b200 import synth


def _case(B=2, C=12, C_a=6, H=11, W=9, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.F32, seed, channel_means=True)
    rng = np.random.default_rng(seed + 50)
    d["w_point"] = rng.uniform(-1, 1, size=(C_a, C_a))
    d["dk"] = rng.uniform(-1, 1, size=(B, C_a, 3, 3))
    return d


def test_p14_identity_mix_is_depthwise_forward(oracle):
    d = _case()
    C_a = 6
    a = oracle.stencil_pw(d["x"], C_a, d["w_large"], np.eye(C_a), d["dk"])
    b = oracle.stencil(d["x"], C_a, d["w_large"], d["dk"])
    assert np.array_equal(a, b)
    fa = oracle.forward_pw(d["x"], C_a, d["w_large"], np.eye(C_a), d["w_dyn"], d["b_dyn"])
    assert np.array_equal(fa, oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"]))


@pytest.mark.parametrize("K", [13, 5])
def test_p15_library_convolutions(oracle, K):
    import torch
    import torch.nn.functional as F

    B, C, C_a, H, W = 2, 20, 16, 17, 21
    d = _case(B, C, C_a, H, W, K, seed=K)
    out = oracle.stencil_pw(d["x"], C_a, d["w_large"], d["w_point"], d["dk"])
    xa = torch.from_numpy(d["x"][:, :C_a].astype(np.float64))
    xm = F.conv2d(xa, torch.from_numpy(d["w_point"]).reshape(C_a, C_a, 1, 1))
    ref = F.conv2d(xm, torch.from_numpy(d["w_large"].astype(np.float64)).reshape(C_a, 1, K, K), padding=K // 2, groups=C_a)
    for b in range(B):
        ref[b] += F.conv2d(xm[b:b + 1], torch.from_numpy(d["dk"][b]).reshape(C_a, 1, 3, 3), padding=1, groups=C_a)[0]
    assert np.allclose(out[:, :C_a], ref.numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(oracle.pointwise(d["x"], C_a, d["w_point"]), xm.numpy(), rtol=1e-13, atol=1e-13)


def test_p16_shared_spatial_kernel_commutes_with_the_mix(oracle):
    B, C, C_a, H, W, K = 1, 8, 5, 10, 12, 7
    d = _case(B, C, C_a, H, W, K, seed=16)
    w_shared = np.broadcast_to(d["w_large"][:1].astype(np.float64), (C_a, K, K)).copy()
    dk_shared = np.broadcast_to(d["dk"][:, :1], (B, C_a, 3, 3)).copy()
    out = oracle.stencil_pw(d["x"], C_a, w_shared, d["w_point"], dk_shared)
    plain = oracle.stencil(d["x"], C_a, w_shared, dk_shared)[:, :C_a]
    want = np.einsum("nk,bkyx->bnyx", d["w_point"], plain)
    assert np.allclose(out[:, :C_a], want, rtol=1e-12, atol=1e-12)
    wrong = np.einsum("kn,bkyx->bnyx", d["w_point"], plain)            # the transposed mix is a different map
    assert np.abs(wrong - want).max() > 1e-2


def test_p17_permutation_and_linearity_in_the_mix(oracle):
    d = _case(seed=17)
    C_a = 6
    perm = np.array([3, 0, 5, 1, 4, 2])
    P = np.zeros((C_a, C_a)); P[np.arange(C_a), perm] = 1.0        # mixed channel n = input channel perm[n]
    out = oracle.stencil_pw(d["x"], C_a, d["w_large"], P, d["dk"])
    xp = d["x"].copy(); xp[:, :C_a] = d["x"][:, perm]
    assert np.array_equal(out[:, :C_a], oracle.stencil(xp, C_a, d["w_large"], d["dk"])[:, :C_a])
    rng = np.random.default_rng(3)
    A, Bm = rng.uniform(-1, 1, (C_a, C_a)), rng.uniform(-1, 1, (C_a, C_a))
    f = lambda M: oracle.stencil_pw(d["x"], C_a, d["w_large"], M, d["dk"])[:, :C_a]
    assert np.allclose(f(2.0 * A - 3.0 * Bm), 2.0 * f(A) - 3.0 * f(Bm), rtol=1e-11, atol=1e-11)


def test_p18_brute_force_tiny(oracle):
    B, C, C_a, H, W, K = 1, 3, 2, 4, 5, 5
    d = _case(B, C, C_a, H, W, K, seed=18)
    out, mag = oracle.stencil_pw(d["x"], C_a, d["w_large"], d["w_point"], d["dk"], want_mag=True)
    x = d["x"].astype(np.float64)
    for c in range(C_a):
        for y in range(H):
            for xx in range(W):
                terms = []
                for i in range(K):
                    for j in range(K):
                        yy, xc = y + i - K // 2, xx + j - K // 2
                        if 0 <= yy < H and 0 <= xc < W:
                            mixed = math.fsum(d["w_point"][c, k] * x[0, k, yy, xc] for k in range(C_a))
                            w = float(d["w_large"][c, i, j])
                            if abs(i - K // 2) <= 1 and abs(j - K // 2) <= 1:
                                w += d["dk"][0, c, i - K // 2 + 1, j - K // 2 + 1]      # ZP(DK) + LK^s
                            terms.append(w * mixed)
                assert out[0, c, y, xx] == pytest.approx(math.fsum(terms), rel=1e-12, abs=1e-12)
                assert mag[0, c, y, xx] >= abs(out[0, c, y, xx]) * (1 - 1e-12)
    assert np.array_equal(out[:, C_a:], x[:, C_a:])


def test_p19_dk_from_unmixed_features_and_identity_channels(oracle):
    B, C, C_a, H, W, K = 2, 10, 4, 9, 8, 5
    d = _case(B, C, C_a, H, W, K, seed=19)
    out, dk = oracle.forward_pw(d["x"], C_a, d["w_large"], d["w_point"], d["w_dyn"], d["b_dyn"], want_dk=True)
    assert np.array_equal(dk, oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"]))
    assert np.array_equal(out, oracle.stencil_pw(d["x"], C_a, d["w_large"], d["w_point"], dk))
    assert np.array_equal(out[:, C_a:], d["x"][:, C_a:].astype(np.float64))
    # changing an identity channel changes nothing in the attention channels
    x2 = d["x"].copy(); x2[:, C_a:] += 1.0
    out2 = oracle.forward_pw(x2, C_a, d["w_large"], d["w_point"], d["w_dyn"], d["b_dyn"])
    assert np.array_equal(out2[:, :C_a], out[:, :C_a])
