"""GPU parity for the backward pass (gradients of the ConvAttn forward of ESC Section 3.3, Eq. 4, one-layer
estimator, depth-wise LK) through the C ABI against the CPU oracle, which is pinned by exact finite differences."""
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
    # B, C, C_a, H, W
    (2, 64, 16, 64, 64),      # one tile per image
    (1, 64, 16, 70, 131),     # several tiles, ragged in both directions
    (3, 24, 8, 9, 11),        # smaller than the kernel, C_a = 8
    (1, 48, 32, 37, 90),      # two channel groups
    (2, 16, 16, 20, 65),      # nothing but attention channels
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_backward(pkg, oracle, shape, dtype, layout):
    import torch

    B, C, C_a, H, W = shape
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(sum(shape) + 1).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    gx = torch.full_like(x, 7.0)
    g_lk = torch.full((C_a, K, K), float("nan"), device="cuda")
    g_w = torch.full((9 * C_a, C_a), float("nan"), device="cuda")
    g_b = torch.full((9 * C_a,), float("nan"), device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    for _ in range(2):                                   # twice: nothing in the workspace may need re-zeroing
        pkg.esc_convattn_backward(x, go_d, C_a, K, wl, wd, bd, gx, g_lk, g_w, g_b, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0

    rx, rlk, rw, rb = oracle.backward(d["x"], go, C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    # scales of the sums: the same gradients of |x|, |go| (every term replaced by its magnitude)
    _, alk, aw, ab = oracle.backward(np.abs(d["x"]), np.abs(go), C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    for name, got, ref, scale in (("w_large", g_lk, rlk, alk), ("w_dyn", g_w, rw, aw), ("b_dyn", g_b, rb, ab)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert (err <= 1e-5 * scale + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"

    got = util.to_host_nchw(gx, layout)
    assert np.array_equal(got[:, C_a:], go[:, C_a:].astype(np.float64)), "identity channels: grad_x must be grad_out"
    # magnitude of the stencil part: |go| through |rotated kernels| = the pinned stencil on magnitudes
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    mag = oracle.stencil(np.abs(go), C_a, np.abs(d["w_large"][:, ::-1, ::-1]).copy(), np.abs(dk[:, :, ::-1, ::-1]).copy())[:, :C_a]
    err = np.abs(got[:, :C_a] - rx[:, :C_a])
    # the constant from the GAP path comes from the fp32 tap gradients: allow their 1e-5 relative noise on its scale
    gg_scale = np.abs(np.einsum("ok,bo->bk", np.abs(d["w_dyn"].astype(np.float64)), np.abs(ab.reshape(1, -1)).repeat(B, 0))) / (H * W)
    bar = 1e-5 * mag + 1e-5 * gg_scale[:, :, None, None] + 1e-30
    if dtype == synth.BF16:
        bar = bar + 2.0 ** -8 * np.abs(rx[:, :C_a]) * 1.001
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"


def _run_backward(pkg, d, go, C_a, K, dtype, layout):
    import torch

    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    B, _, H, W = d["x"].shape
    gx = torch.full_like(x, 7.0)
    g_lk = torch.full((C_a, K, K), float("nan"), device="cuda")
    g_w = torch.full((9 * C_a, C_a), float("nan"), device="cuda")
    g_b = torch.full((9 * C_a,), float("nan"), device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    for _ in range(2):
        pkg.esc_convattn_backward(x, go_d, C_a, K, wl, wd, bd, gx, g_lk, g_w, g_b, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    return gx, g_lk, g_w, g_b


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("shape", [(1, 64, 16, 300, 640), (6, 32, 32, 130, 200), (40, 16, 16, 64, 64), (2, 32, 16, 45, 72)], ids=lambda s: "x".join(map(str, s)))
def test_backward_weight_gradients_many_units(pkg, oracle, shape, layout):
    """bf16 (both layouts; W a multiple of 8 as the NCHW kernel wants), where the tap gradients run on the tensor cores: 190, 432 and 160 units of 64x16 on 148 SMs, so CTAs
    walk two or three units (staging buffers, planes and barriers are re-used; image and channel group change inside
    a walk); the three weight gradients against the oracle, and against the FP32-pipe kernels."""
    B, C, C_a, H, W = shape
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + 3, per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(sum(shape) + 4).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    _, g_lk, g_w, g_b = _run_backward(pkg, d, go, C_a, K, synth.BF16, layout)
    _, rlk, rw, rb = oracle.backward(d["x"], go, C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    _, alk, aw, ab = oracle.backward(np.abs(d["x"]), np.abs(go), C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    for name, got, ref, scale in (("w_large", g_lk, rlk, alk), ("w_dyn", g_w, rw, aw), ("b_dyn", g_b, rb, ab)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert (err <= 1e-5 * scale + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"
    pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
    try:
        _, f_lk, f_w, f_b = _run_backward(pkg, d, go, C_a, K, synth.BF16, layout)
    finally:
        pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)
    for name, a, b, scale in (("w_large", g_lk, f_lk, alk), ("w_dyn", g_w, f_w, aw), ("b_dyn", g_b, f_b, ab)):
        err = np.abs(a.cpu().numpy().astype(np.float64) - b.cpu().numpy().astype(np.float64))
        assert (err <= 2e-5 * scale + 1e-30).all(), f"grad {name}: the two kernels differ by {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("K", [9, 5, 3])
def test_backward_smaller_large_kernels(pkg, oracle, K, dtype, layout):
    """K < 13: the tap-gradient kernels form the 13 x 13 taps' gradients, of which the K x K in the middle are the large
    kernel's; grad_x runs the K x K stencil.  All four gradients against the oracle at the true K."""
    B, C, C_a, H, W = 2, 32, 16, 37, 72
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=100 + K, per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(200 + K).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    gx, g_lk, g_w, g_b = _run_backward(pkg, d, go, C_a, K, dtype, layout)
    rx, rlk, rw, rb = oracle.backward(d["x"], go, C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    _, alk, aw, ab = oracle.backward(np.abs(d["x"]), np.abs(go), C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    assert tuple(g_lk.shape) == (C_a, K, K)
    for name, got, ref, scale in (("w_large", g_lk, rlk, alk), ("w_dyn", g_w, rw, aw), ("b_dyn", g_b, rb, ab)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert (err <= 1e-5 * scale + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"
    got = util.to_host_nchw(gx, layout)
    assert np.array_equal(got[:, C_a:], go[:, C_a:].astype(np.float64))
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    mag = oracle.stencil(np.abs(go), C_a, np.abs(d["w_large"][:, ::-1, ::-1]).copy(), np.abs(dk[:, :, ::-1, ::-1]).copy())[:, :C_a]
    gg_scale = np.abs(np.einsum("ok,bo->bk", np.abs(d["w_dyn"].astype(np.float64)), np.abs(ab.reshape(1, -1)).repeat(B, 0))) / (H * W)
    bar = 1e-5 * mag + 1e-5 * gg_scale[:, :, None, None] + 1e-30
    if dtype == synth.BF16:
        bar = bar + 2.0 ** -8 * np.abs(rx[:, :C_a]) * 1.001
    err = np.abs(got[:, :C_a] - rx[:, :C_a])
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"


def test_backward_rejections(pkg):
    import torch

    x = torch.zeros(1, 8, 8, 16, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(16, 15, 15, dtype=torch.bfloat16, device="cuda")
    assert pkg.esc_convattn_backward_workspace_bytes(1, 16, 8, 8, 15) == 0         # K = 3 .. 13 only
    assert pkg.esc_convattn_backward_workspace_bytes(1, 16, 8, 8, 9) > 0
    L = pkg.lib()
    ws = pkg.new_backward_workspace(1, 16, 8, 8, 13)
    rc = L.esc_convattn_backward(x.data_ptr(), x.data_ptr(), 1, 16, 16, 8, 8, 15, w.data_ptr(), w.data_ptr(), w.data_ptr(),
                                 x.data_ptr(), None, None, None, 1, 1, ws.data_ptr(), ws.numel(), None)
    assert rc == 3

@pytest.mark.parametrize("layout", LAYOUTS)
def test_backward_full_size_640x360(pkg, oracle, layout):
    """The size bench.py times (1 x 64 x 360 x 640, C_a = 16, K = 13, bf16), every gradient element against the oracle:
    230 units of 64x16 on 148 SMs for the tap gradients and the stencil pass."""
    B, C, C_a, H, W, K = 1, 64, 16, 360, 640, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=640360, per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(640361).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    gx, g_lk, g_w, g_b = _run_backward(pkg, d, go, C_a, K, synth.BF16, layout)
    rx, rlk, rw, rb = oracle.backward(d["x"], go, C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    _, alk, aw, ab = oracle.backward(np.abs(d["x"]), np.abs(go), C_a, d["w_large"], d["w_dyn"], d["b_dyn"])
    for name, got, ref, scale in (("w_large", g_lk, rlk, alk), ("w_dyn", g_w, rw, aw), ("b_dyn", g_b, rb, ab)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
        assert (err <= 1e-5 * scale + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"
    got = util.to_host_nchw(gx, layout)
    assert np.array_equal(got[:, C_a:], go[:, C_a:].astype(np.float64))
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    mag = oracle.stencil(np.abs(go), C_a, np.abs(d["w_large"][:, ::-1, ::-1]).copy(), np.abs(dk[:, :, ::-1, ::-1]).copy())[:, :C_a]
    gg_scale = np.abs(np.einsum("ok,bo->bk", np.abs(d["w_dyn"].astype(np.float64)), np.abs(ab.reshape(1, -1)).repeat(B, 0))) / (H * W)
    err = np.abs(got[:, :C_a] - rx[:, :C_a])
    bar = 1e-5 * mag + 1e-5 * gg_scale[:, :, None, None] + 2.0 ** -8 * np.abs(rx[:, :C_a]) * 1.001 + 1e-30
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"
