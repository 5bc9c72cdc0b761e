"""Pins for the oracle's dense large kernel (ESC paper, Section 3.2: LK in R^{13x13x16x16}, used in Eq. 4 line 3).

P20  a dense kernel that is diagonal in (output, input) channel is the pinned depth-wise stencil, bit for bit
P21  library route: torch fp64 dense conv2d plus a depth-wise conv2d for the dynamic kernel
P22  a kernel that factors as w_dense[n,k] = M[n,k] * w[k] is "depth-wise, then point-wise": out = M applied per
     pixel to the pinned depth-wise result (tells (n,k) from (k,n))
P23  pure-Python brute force on a tiny map, borders included; identity channels pass through
"""
import math

import numpy as np
import pytest

from paper_2503_06671_b200 import synth


def _case(B=2, C=9, C_a=5, H=8, W=10, K=5, seed=0):
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.F32, seed, channel_means=True)
    rng = np.random.default_rng(seed + 90)
    d["w_dense"] = rng.uniform(-1, 1, size=(C_a, C_a, K, K))
    d["dk"] = rng.uniform(-1, 1, size=(B, C_a, 3, 3))
    return d


def test_p20_diagonal_dense_kernel_is_the_depthwise_stencil(oracle):
    d = _case()
    C_a, K = 5, 5
    wd = np.zeros((C_a, C_a, K, K))
    for c in range(C_a):
        wd[c, c] = d["w_large"][c]
    assert np.array_equal(oracle.stencil_dense(d["x"], C_a, wd, d["dk"]), oracle.stencil(d["x"], C_a, d["w_large"], d["dk"]))


@pytest.mark.parametrize("K", [13, 3])
def test_p21_library_dense_convolution(oracle, K):
    import torch
    import torch.nn.functional as F

    B, C, C_a, H, W = 2, 20, 16, 15, 18
    d = _case(B, C, C_a, H, W, K, seed=K)
    out = oracle.stencil_dense(d["x"], C_a, d["w_dense"], d["dk"])
    xa = torch.from_numpy(d["x"][:, :C_a].astype(np.float64))
    ref = F.conv2d(xa, torch.from_numpy(d["w_dense"]), padding=K // 2)
    for b in range(B):
        ref[b] += F.conv2d(xa[b:b + 1], torch.from_numpy(d["dk"][b]).reshape(C_a, 1, 3, 3), padding=1, groups=C_a)[0]
    assert np.allclose(out[:, :C_a], ref.numpy(), rtol=1e-12, atol=1e-12)
    assert np.array_equal(out[:, C_a:], d["x"][:, C_a:].astype(np.float64))


def test_p22_factored_kernel_is_depthwise_then_pointwise(oracle):
    B, C, C_a, H, W, K = 1, 7, 4, 9, 11, 7
    d = _case(B, C, C_a, H, W, K, seed=22)
    M = np.random.default_rng(22).uniform(-1, 1, size=(C_a, C_a))
    w = d["w_large"].astype(np.float64)                                   # [k, K, K]
    wd = M[:, :, None, None] * w[None, :, :, :]
    zero_dk = np.zeros((B, C_a, 3, 3))
    out = oracle.stencil_dense(d["x"], C_a, wd, zero_dk)
    dw = oracle.stencil(d["x"], C_a, w, zero_dk)[:, :C_a]
    want = np.einsum("nk,bkyx->bnyx", M, dw)
    assert np.allclose(out[:, :C_a], want, rtol=1e-12, atol=1e-12)
    assert np.abs(np.einsum("kn,bkyx->bnyx", M, dw) - want).max() > 1e-2   # the transposed reading differs


def test_p23_brute_force_tiny(oracle):
    B, C, C_a, H, W, K = 1, 3, 2, 4, 5, 3
    d = _case(B, C, C_a, H, W, K, seed=23)
    out, mag = oracle.stencil_dense(d["x"], C_a, d["w_dense"], d["dk"], want_mag=True)
    x = d["x"].astype(np.float64)
    for n in range(C_a):
        for y in range(H):
            for xx in range(W):
                terms = []
                for i in range(K):
                    for j in range(K):
                        yy, xc = y + i - K // 2, xx + j - K // 2
                        if 0 <= yy < H and 0 <= xc < W:
                            for k in range(C_a):
                                terms.append(d["w_dense"][n, k, i, j] * x[0, k, yy, xc])
                            terms.append(d["dk"][0, n, i, j] * x[0, n, yy, xc])    # K = 3: the same nine taps
                assert out[0, n, y, xx] == pytest.approx(math.fsum(terms), rel=1e-12, abs=1e-12)
                assert mag[0, n, y, xx] == pytest.approx(math.fsum(abs(t) for t in terms), rel=1e-12)
    assert np.array_equal(out[:, C_a:], x[:, C_a:])
    fwd, dk = oracle.forward_dense(d["x"], C_a, d["w_dense"], d["w_dyn"], d["b_dyn"], want_dk=True)
    assert np.array_equal(dk, oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"]))
    assert np.array_equal(fwd, oracle.stencil_dense(d["x"], C_a, d["w_dense"], dk))
