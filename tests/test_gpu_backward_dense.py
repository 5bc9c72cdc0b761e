"""GPU parity for the backward pass with the dense large kernel (ESC Section 3.2) through the C ABI against the CPU
oracle, which is pinned by exact differences of the pinned dense forward.

Bars: every gradient is a sum of products; `scale` is the same sum with every factor replaced by its magnitude (the
oracle run on |x|, |go|, |weights|).  Weight gradients (fp32 accumulation of exact products): 1e-5 * scale.  grad_x:
1e-5 * scale (5e-5 on the tensor cores), and for bf16 tensors two roundings of the result (the stencil pass stores it, the estimator's constant is
added to the stored value): 2^-8 * (|reference - constant| + |reference|) more (a bf16 rounding moves a value by at most 2^-8 of it).
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

LAYOUTS = [synth.NCHW, synth.NHWC]
DTYPES = [synth.F32, synth.BF16]
NAMES = ("w_dense", "w_dyn", "b_dyn")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


def _run(pkg, d, wdn, go, C_a, K, dtype, layout):
    import torch

    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    _, wd, bd = util.weights_to_device(d, dtype)
    wdn_d = torch.from_numpy(wdn).to("cuda", util.torch_dtype(dtype))
    B, _, H, W = d["x"].shape
    gx = torch.full_like(x, 7.0)
    g = {"w_dense": torch.full((C_a, C_a, K, K), float("nan"), device="cuda"),
         "w_dyn": torch.full((9 * C_a, C_a), float("nan"), device="cuda"),
         "b_dyn": torch.full((9 * C_a,), float("nan"), device="cuda")}
    ws = pkg.new_backward_dense_workspace(B, C_a, H, W, K)
    for _ in range(2):                                   # twice: nothing in the workspace may need re-zeroing
        pkg.esc_convattn_backward_dense(x, go_d, C_a, K, wdn_d, wd, bd, gx, g["w_dense"], g["w_dyn"], g["b_dyn"],
                                        util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    return util.to_host_nchw(gx, layout), {k: v.cpu().numpy().astype(np.float64) for k, v in g.items()}


def _check(oracle, d, wdn, go, C_a, dtype, gx, g):
    B = d["x"].shape[0]
    ref = oracle.backward_dense(d["x"], go, C_a, wdn, d["w_dyn"], d["b_dyn"])
    mag = oracle.backward_dense(np.abs(d["x"]), np.abs(go), C_a, np.abs(wdn), np.abs(d["w_dyn"]), np.abs(d["b_dyn"]))
    for name, r, a in zip(NAMES, ref[1:], mag[1:]):
        err = np.abs(g[name] - r)
        assert (err <= 1e-5 * a + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(a, 1e-30)).max():.3e} of its scale"
    rx, ax = ref[0], mag[0]
    assert np.array_equal(gx[:, C_a:], go[:, C_a:].astype(np.float64)), "identity channels: grad_x must be grad_out"
    err = np.abs(gx[:, :C_a] - rx[:, :C_a])
    # bf16: the stencil pass is the forward's tensor-core kernel, whose accumulation (16 products and the running sum per
    # step, 170 steps) is within 5e-5 of the magnitudes involved -- the forward's parity bar
    bar = (5e-5 if dtype == synth.BF16 else 1e-5) * ax[:, :C_a] + 1e-30
    if dtype == synth.BF16:
        # the estimator's constant: the whole gradient minus the one with the generator frozen at this input's dk
        # (the dynamic kernel is depth-wise, so the pinned depth-wise backward with a zero large kernel has the same constant)
        dk = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
        z = np.zeros((C_a, wdn.shape[-1], wdn.shape[-1]))
        const = np.stack([(oracle.backward(d["x"][i:i + 1], go[i:i + 1], C_a, z, d["w_dyn"], d["b_dyn"])[0]
                           - oracle.backward(d["x"][i:i + 1], go[i:i + 1], C_a, z, np.zeros_like(d["w_dyn"]), dk[i].reshape(-1))[0])[0, :C_a, :1, :1]
                          for i in range(B)])
        bar = bar + 2.0 ** -8 * (np.abs(rx[:, :C_a] - const) + np.abs(rx[:, :C_a])) * 1.01   # the stencil part's rounding, then the sum's
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"


SHAPES = [
    # B, C, C_a, H, W, K
    (2, 48, 16, 64, 64, 13),     # training patches: eight tiles of 32 x 16 per image
    (1, 64, 16, 37, 90, 13),     # ragged in both directions
    (1, 16, 16, 9, 11, 13),      # smaller than the kernel, nothing but attention channels
    (1, 32, 16, 29, 31, 9),      # K = 9: the middle of the 13 x 13 sums
    (1, 32, 16, 20, 24, 3),      # K = 3
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_backward_dense(pkg, oracle, shape, dtype, layout):
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), per_image_scale=True, channel_means=True)
    wdn = synth.make_dense_kernel(C_a, K, dtype, seed=sum(shape))
    go = synth.round_to(np.random.default_rng(sum(shape) + 1).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    gx, g = _run(pkg, d, wdn, go, C_a, K, dtype, layout)
    _check(oracle, d, wdn, go, C_a, dtype, gx, g)


def test_backward_dense_many_tiles(pkg, oracle):
    """More tiles than blocks: 3 x 13 x 7 = 273 tiles of 32 x 16 on one block per SM, so blocks add up two tiles, some of
    them of two images, in their registers; bf16 NHWC, where the weight gradient is a matrix product per tap on the tensor
    cores and grad_x runs on the tcgen05 kernel."""
    shape = (3, 32, 16, 200, 200, 13)
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=91, per_image_scale=True, channel_means=True)
    wdn = synth.make_dense_kernel(C_a, K, synth.BF16, seed=91)
    go = synth.round_to(np.random.default_rng(92).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    gx, g = _run(pkg, d, wdn, go, C_a, K, synth.BF16, synth.NHWC)
    _check(oracle, d, wdn, go, C_a, synth.BF16, gx, g)
    # the FP32-pipe kernel on the same bf16 tensors (what fp32 tensors always use): the same sums in another order
    pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
    try:
        _, g2 = _run(pkg, d, wdn, go, C_a, K, synth.BF16, synth.NHWC)
    finally:
        pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)
    mag = oracle.backward_dense(np.abs(d["x"]), np.abs(go), C_a, np.abs(wdn), np.abs(d["w_dyn"]), np.abs(d["b_dyn"]))[1]
    assert (np.abs(g2["w_dense"] - g["w_dense"]) <= 2e-5 * mag).all()


def test_diagonal_kernel_equals_the_depthwise_backward(pkg):
    """A dense kernel that is zero off the diagonal is the depth-wise form: g_W_dyn and g_b_dyn must be what
    esc_convattn_backward returns bit for bit (same kernels), the diagonal of g_w_dense its g_LK to fp32 noise."""
    import torch

    B, C, C_a, H, W, K = 2, 32, 16, 45, 72, 13
    dtype, layout = synth.BF16, synth.NHWC
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=5, per_image_scale=True, channel_means=True)
    go = synth.round_to(np.random.default_rng(6).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    wdn = np.zeros((C_a, C_a, K, K), dtype=np.float32)
    for c in range(C_a):
        wdn[c, c] = d["w_large"][c]
    gx, g = _run(pkg, d, wdn, go, C_a, K, dtype, layout)
    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    gx1 = torch.full_like(x, 7.0)
    g_lk = torch.empty((C_a, K, K), device="cuda"); g_w = torch.empty((9 * C_a, C_a), device="cuda"); g_b = torch.empty((9 * C_a,), device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_backward(x, go_d, C_a, K, wl, wd, bd, gx1, g_lk, g_w, g_b, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert np.array_equal(g["w_dyn"], g_w.cpu().numpy().astype(np.float64))
    assert np.array_equal(g["b_dyn"], g_b.cpu().numpy().astype(np.float64))
    lk = g_lk.cpu().numpy().astype(np.float64)
    diag = np.stack([g["w_dense"][c, c] for c in range(C_a)])
    np.testing.assert_allclose(diag, lk, rtol=1e-4, atol=1e-5 * np.abs(lk).max())


def test_backward_dense_rejections(pkg):
    import torch

    B, C, C_a, H, W, K = 1, 32, 8, 16, 16, 13                         # the dense kernel is 16 x 16 channels
    x = torch.zeros((B, H, W, C), device="cuda", dtype=torch.bfloat16)
    gx = torch.zeros_like(x)
    wdn = torch.zeros((C_a, C_a, K, K), device="cuda", dtype=torch.bfloat16)
    wd = torch.zeros((9 * C_a, C_a), device="cuda", dtype=torch.bfloat16)
    bd = torch.zeros((9 * C_a,), device="cuda", dtype=torch.bfloat16)
    assert pkg.esc_convattn_backward_dense_workspace_bytes(B, C_a, H, W, K) == 0
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_backward_dense(x, x.clone(), C_a, K, wdn, wd, bd, gx, None, None, None, util.layout_code(synth.NHWC), ws)
    assert e.value.status == 3
    # the depth-wise workspace is too small for it
    C_a = 16
    wdn = torch.zeros((C_a, C_a, K, K), device="cuda", dtype=torch.bfloat16)
    wd = torch.zeros((9 * C_a, C_a), device="cuda", dtype=torch.bfloat16)
    bd = torch.zeros((9 * C_a,), device="cuda", dtype=torch.bfloat16)
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_backward_dense(x, x.clone(), C_a, K, wdn, wd, bd, gx, None, None, None, util.layout_code(synth.NHWC), ws)
    assert e.value.status == 6

def test_backward_dense_weight_gradient_full_size_640x360(pkg, oracle):
    """The size bench.py times (1 x 64 x 360 x 640, C_a = 16, K = 13, bf16 NHWC; 920 tiles on one block per SM): 400 sampled
    entries of the 43,264 of the kernel's gradient against the oracle, entry by entry."""
    B, C, C_a, H, W, K = 1, 64, 16, 360, 640, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=640360, per_image_scale=True, channel_means=True)
    wdn = synth.make_dense_kernel(C_a, K, synth.BF16, seed=640360)
    go = synth.round_to(np.random.default_rng(640361).standard_normal(size=d["x"].shape).astype(np.float32), synth.BF16)
    _, g = _run(pkg, d, wdn, go, C_a, K, synth.BF16, synth.NHWC)
    rng = np.random.default_rng(5)
    idx = np.unique(np.concatenate([rng.integers(0, C_a * C_a * K * K, size=392),
                                    np.array([0, K * K - 1, C_a * C_a * K * K - 1, (5 * C_a + 5) * K * K + 84,   # corners, a centre tap
                                              (0 * C_a + 15) * K * K + 12, (15 * C_a + 0) * K * K + 156])]))
    vals, mags = oracle.backward_dense_points(d["x"], go, C_a, K, idx)
    got = g["w_dense"].reshape(-1)[idx]
    err = np.abs(got - vals)
    assert (err <= 1e-5 * mags + 1e-30).all(), f"grad w_dense: worst {(err / np.maximum(mags, 1e-30)).max():.3e} of its scale"
