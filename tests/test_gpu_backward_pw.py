"""GPU parity for the backward pass of the decomposed form (ESC Eq. 5: point-wise LK^c in front of the depth-wise stage)
through the C ABI against the CPU oracle, which is pinned by exact differences of the pinned forward.

Bars.  Every gradient is a sum of products; `scale` is the same sum with every factor replaced by its magnitude (the
oracle run on |x|, |go|, |weights|).  fp32 tensors: 1e-5 * scale (fp32 accumulation in another order).  bf16 tensors keep
the mixed features m and dL/dm in bf16, as a bf16 network stores every feature map: a rounding moves a term by at
most 2^-8 of its magnitude, so the worst case of the two is 2^-7 * scale; the test asks for half of that,
(1e-5 + 2^-8) * scale (the roundings are neither all worst-case nor all of one sign).  Because any such bar is wide for
long sums, the error is also bounded in the Euclidean norm (2^-7 of the reference's), which a wrong index or a transposed
operand misses at any size.
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

LAYOUTS = [synth.NCHW, synth.NHWC]
DTYPES = [synth.F32, synth.BF16]
NAMES = ("w_large", "w_point", "w_dyn", "b_dyn")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


def _run(pkg, d, wp, go, C_a, K, dtype, layout, twice=True):
    import torch

    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    wp_d = torch.from_numpy(wp).to("cuda", util.torch_dtype(dtype))
    B, _, H, W = d["x"].shape
    gx = torch.full_like(x, 7.0)
    g = {"w_large": torch.full((C_a, K, K), float("nan"), device="cuda"),
         "w_point": torch.full((C_a, C_a), float("nan"), device="cuda"),
         "w_dyn": torch.full((9 * C_a, C_a), float("nan"), device="cuda"),
         "b_dyn": torch.full((9 * C_a,), float("nan"), device="cuda")}
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    for _ in range(2 if twice else 1):                   # twice: nothing in the workspace may need re-zeroing
        pkg.esc_convattn_backward_pw(x, go_d, C_a, K, wl, wp_d, wd, bd, gx, g["w_large"], g["w_point"], g["w_dyn"], g["b_dyn"],
                                     util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    return util.to_host_nchw(gx, layout), {k: v.cpu().numpy().astype(np.float64) for k, v in g.items()}


def _check(oracle, d, wp, go, C_a, dtype, gx, g):
    ref = oracle.backward_pw(d["x"], go, C_a, d["w_large"], wp, d["w_dyn"], d["b_dyn"])
    mag = oracle.backward_pw(np.abs(d["x"]), np.abs(go), C_a, np.abs(d["w_large"]), np.abs(wp), np.abs(d["w_dyn"]), np.abs(d["b_dyn"]))
    rx, ax = ref[0], mag[0]
    rel = 1e-5 + (2.0 ** -8 if dtype == synth.BF16 else 0.0)
    for name, r, a in zip(NAMES, ref[1:], mag[1:]):
        err = np.abs(g[name] - r)
        assert (err <= rel * a + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(a, 1e-30)).max():.3e} of its scale"
        if dtype == synth.BF16:
            assert np.linalg.norm(err) <= 2.0 ** -7 * np.linalg.norm(r) + 1e-30, f"grad {name}: {np.linalg.norm(err) / np.linalg.norm(r):.3e} in norm"
    assert np.array_equal(gx[:, C_a:], go[:, C_a:].astype(np.float64)), "identity channels: grad_x must be grad_out"
    err = np.abs(gx[:, :C_a] - rx[:, :C_a])
    bar = rel * ax[:, :C_a] + 1e-30
    if dtype == synth.BF16:
        bar = bar + 2.0 ** -8 * np.abs(rx[:, :C_a]) * 1.001       # the result's own rounding
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"
    if dtype == synth.BF16:
        assert np.linalg.norm(err) <= 2.0 ** -7 * np.linalg.norm(rx[:, :C_a])


SHAPES = [
    # B, C, C_a, H, W, K
    (2, 48, 16, 64, 64, 13),     # ESC-FP width, training patches: four chunks of pixels per image
    (1, 64, 16, 70, 136, 13),    # several tiles, ragged last chunk
    (3, 24, 8, 9, 11, 13),       # smaller than the kernel, C_a = 8, less than one pass of pixels
    (1, 48, 32, 37, 88, 13),     # C_a = 32: two channel groups, four (n, k) pairs per thread
    (2, 16, 16, 20, 65, 13),     # nothing but attention channels
    (1, 12, 4, 33, 35, 5),       # C_a = 4, K = 5, rows that are not 16-byte multiples
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_backward_pw(pkg, oracle, shape, dtype, layout):
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), per_image_scale=True, channel_means=True)
    wp = synth.make_pointwise(C_a, dtype, seed=sum(shape))
    go = synth.round_to(np.random.default_rng(sum(shape) + 1).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    gx, g = _run(pkg, d, wp, go, C_a, K, dtype, layout)
    _check(oracle, d, wp, go, C_a, dtype, gx, g)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_backward_pw_many_units(pkg, oracle, layout):
    """bf16 at a size where the tap-gradient and stencil kernels walk several units per CTA and the per-pixel kernels
    run 188 chunks; also against the FP32-pipe kernels."""
    shape = (1, 64, 16, 300, 640, 13)
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=77, per_image_scale=True, channel_means=True)
    wp = synth.make_pointwise(C_a, synth.BF16, seed=77)
    go = synth.round_to(np.random.default_rng(78).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    gx, g = _run(pkg, d, wp, go, C_a, K, synth.BF16, layout)
    _check(oracle, d, wp, go, C_a, synth.BF16, gx, g)
    pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
    try:
        gx2, g2 = _run(pkg, d, wp, go, C_a, K, synth.BF16, layout, twice=False)
    finally:
        pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)
    _check(oracle, d, wp, go, C_a, synth.BF16, gx2, g2)


def test_identity_mix_equals_the_depthwise_backward(pkg, oracle):
    """With LK^c = I the mixed features are x itself (no rounding), so every gradient must equal what
    esc_convattn_backward returns, to fp32 summation noise."""
    import torch

    B, C, C_a, H, W, K = 2, 32, 16, 45, 72, 13
    dtype, layout = synth.BF16, synth.NHWC
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=5, per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(6).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    gx, g = _run(pkg, d, np.eye(C_a, dtype=np.float32), go, C_a, K, dtype, layout)
    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    gx1 = torch.full_like(x, 7.0)
    g_lk = torch.empty((C_a, K, K), device="cuda"); g_w = torch.empty((9 * C_a, C_a), device="cuda"); g_b = torch.empty((9 * C_a,), device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_backward(x, go_d, C_a, K, wl, wd, bd, gx1, g_lk, g_w, g_b, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert np.array_equal(g["w_large"], g_lk.cpu().numpy().astype(np.float64))
    assert np.array_equal(g["b_dyn"], g_b.cpu().numpy().astype(np.float64))
    ref_w = g_w.cpu().numpy().astype(np.float64)                     # the image means are added up in another order
    np.testing.assert_allclose(g["w_dyn"], ref_w, rtol=1e-5, atol=1e-6 * np.abs(ref_w).max())
    # grad_x: here the estimator's constant is added behind a rounding of dL/dm, there in front of the only rounding;
    # the constant itself from the oracle (the whole gradient minus the one with the generator frozen)
    a, b = gx, util.to_host_nchw(gx1, layout)
    dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
    const = np.stack([(oracle.backward(d["x"][i:i + 1], go[i:i + 1], C_a, d["w_large"], d["w_dyn"], d["b_dyn"])[0]
                       - oracle.backward(d["x"][i:i + 1], go[i:i + 1], C_a, d["w_large"], np.zeros_like(d["w_dyn"]), dk[i].reshape(-1))[0])[0, :C_a, :1, :1]
                      for i in range(B)])
    assert np.array_equal(a[:, C_a:], b[:, C_a:])
    assert (np.abs(a - b)[:, :C_a] <= 2.0 ** -7 * (np.abs(b[:, :C_a]) + np.abs(const)) + 1e-6).all()


def test_backward_pw_rejections(pkg):
    import torch

    B, C, C_a, H, W, K = 1, 24, 12, 16, 16, 13                        # C_a = 12 has no instantiation
    x = torch.zeros((B, H, W, C), device="cuda", dtype=torch.bfloat16)
    gx = torch.zeros_like(x)
    wl = torch.zeros((C_a, K, K), device="cuda", dtype=torch.bfloat16)
    wp = torch.zeros((C_a, C_a), device="cuda", dtype=torch.bfloat16)
    wd = torch.zeros((9 * C_a, C_a), device="cuda", dtype=torch.bfloat16)
    bd = torch.zeros((9 * C_a,), device="cuda", dtype=torch.bfloat16)
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_backward_pw(x, x.clone(), C_a, K, wl, wp, wd, bd, gx, None, None, None, None, util.layout_code(synth.NHWC), ws)
    assert e.value.status == 3

def test_backward_pw_full_size_640x360(pkg, oracle):
    """The size bench.py times (1 x 64 x 360 x 640, C_a = 16, K = 13, bf16 NHWC): 450 chunks of pixels per per-pixel kernel."""
    shape = (1, 64, 16, 360, 640, 13)
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=640360, per_image_scale=True, channel_means=True)
    wp = synth.make_pointwise(C_a, synth.BF16, seed=640360)
    go = synth.round_to(np.random.default_rng(640361).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    gx, g = _run(pkg, d, wp, go, C_a, K, synth.BF16, synth.NHWC)
    _check(oracle, d, wp, go, C_a, synth.BF16, gx, g)
