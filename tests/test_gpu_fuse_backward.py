"""GPU parity for the backward pass of Conv_fuse (ESC Eq. 4 line 4 with the residual of Eq. 3 line 3) through the C ABI
against the CPU oracle, which is pinned by exact differences of the pinned forward.

Bars: g_W, g_b are fp32 sums of exact products (bf16) or fp32 products: 1e-5 of the sums' scale (the same sums of
magnitudes).  g_cat: 1e-5 of its scale (5e-5 on the tensor cores) plus, for bf16, the rounding of the result,
2^-8 * |reference|.
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

LAYOUTS = [synth.NCHW, synth.NHWC]
DTYPES = [synth.F32, synth.BF16]


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


SHAPES = [
    # B, C, H, W
    (2, 64, 64, 64),      # the main model's width, training patches
    (1, 48, 37, 88),      # ESC-FP's width, ragged run of pixels
    (3, 32, 9, 11),       # less than one pass of pixels per image; runs cross images
    (1, 16, 20, 24),      # the narrow case: 16 tiles x 16 slices
    (1, 64, 130, 200),    # several passes per block
    (1, 64, 360, 640),    # the size bench.py times: seven runs of 256 pixels per block, 129 blocks
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_fuse_backward(pkg, oracle, shape, dtype, layout):
    import torch

    B, C, H, W = shape
    rng = np.random.default_rng(sum(shape))
    cat = synth.round_to(rng.standard_normal((B, C, H, W)).astype(np.float32) + 0.25, dtype)
    go = synth.round_to(rng.standard_normal((B, C, H, W)).astype(np.float32), dtype)
    w = synth.make_fuse(C, dtype, seed=sum(shape))["w_fuse"]
    tdt = util.torch_dtype(dtype)
    cat_d = util.to_device(cat, dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    w_d = torch.from_numpy(w).to("cuda", tdt)
    g_cat = torch.full_like(cat_d, 7.0)
    g_w = torch.full((C, C), float("nan"), device="cuda")
    g_b = torch.full((C,), float("nan"), device="cuda")
    for _ in range(2):
        pkg.esc_conv_fuse_backward(cat_d, go_d, w_d, g_cat, g_w, g_b, util.layout_code(layout))
    torch.cuda.synchronize()
    r_cat, r_w, r_b, m_cat = oracle.fuse_backward(cat, go, w, want_mag=True)
    _, a_w, a_b = oracle.fuse_backward(np.abs(cat), np.abs(go), np.abs(w))
    err = np.abs(g_w.cpu().numpy().astype(np.float64) - r_w)
    assert (err <= 1e-5 * a_w + 1e-30).all(), f"grad W_fuse: worst {(err / a_w).max():.3e} of its scale"
    err = np.abs(g_b.cpu().numpy().astype(np.float64) - r_b)
    assert (err <= 1e-5 * a_b + 1e-30).all(), f"grad b_fuse: worst {(err / a_b).max():.3e} of its scale"
    got = util.to_host_nchw(g_cat, layout)
    err = np.abs(got - r_cat)
    bar = (5e-5 if dtype == synth.BF16 else 1e-5) * m_cat + 1e-30
    if dtype == synth.BF16:
        bar = bar + 2.0 ** -8 * np.abs(r_cat) * 1.001
    assert (err <= bar).all(), f"grad cat: {int((err > bar).sum())} values beyond the bound"


def test_fuse_backward_optional_outputs_and_rejections(pkg, oracle):
    import torch

    B, C, H, W = 1, 64, 24, 40
    rng = np.random.default_rng(3)
    cat = synth.round_to(rng.standard_normal((B, C, H, W)).astype(np.float32), synth.BF16)
    go = synth.round_to(rng.standard_normal((B, C, H, W)).astype(np.float32), synth.BF16)
    w = synth.make_fuse(C, synth.BF16, seed=3)["w_fuse"]
    cat_d = util.to_device(cat, synth.BF16, synth.NHWC); go_d = util.to_device(go, synth.BF16, synth.NHWC)
    w_d = torch.from_numpy(w).to("cuda", torch.bfloat16)
    g_cat = torch.full_like(cat_d, 7.0)
    lc = util.layout_code(synth.NHWC)
    pkg.esc_conv_fuse_backward(cat_d, go_d, w_d, g_cat, None, None, lc)          # no weight gradients: the 1x1 kernel alone
    torch.cuda.synchronize()
    r_cat, _, _, m_cat = oracle.fuse_backward(cat, go, w, want_mag=True)
    err = np.abs(util.to_host_nchw(g_cat, synth.NHWC) - r_cat)
    assert (err <= 5e-5 * m_cat + 2.0 ** -8 * np.abs(r_cat) * 1.001).all()
    with pytest.raises(pkg.EscError) as e:                                         # grad_cat over grad_out
        pkg.esc_conv_fuse_backward(cat_d, go_d, w_d, go_d, None, None, lc)
    assert e.value.status == 5
    x40 = torch.zeros((1, 8, 8, 40), device="cuda", dtype=torch.bfloat16)          # C = 40 has no instantiation
    assert pkg.esc_conv_fuse_backward_workspace_bytes(1, 40, 8, 8) == 0
    with pytest.raises(pkg.EscError):
        pkg.esc_conv_fuse_backward(x40, x40.clone(), torch.zeros((40, 40), device="cuda", dtype=torch.bfloat16), torch.zeros_like(x40), None, None, lc)
