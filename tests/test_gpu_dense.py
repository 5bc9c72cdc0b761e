"""GPU parity for the dense large kernel (ESC paper, Section 3.2: LK in R^{13x13x16x16}, in Eq. 4 line 3),
through the C ABI against the CPU oracle."""
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


def _check(got, ref, mag, dtype, C_a, what):
    err = np.abs(got[:, :C_a] - ref[:, :C_a])
    if dtype == synth.F32:
        # 16 * K * K + 9 fp32 FMAs in a row: rounding noise grows like the square root of the count
        bar = 1e-5 * mag + 1e-30
    else:
        # bf16 products are exact in fp32; the tensor cores add 16 of them and the running sum per step
        # (170 steps, each within 2^-23 of the magnitudes involved), then one rounding of the result to bf16
        bar = 2.0 ** -8 * np.abs(ref[:, :C_a]) * 1.001 + 5e-5 * mag + 1e-30
    assert (err <= bar).all(), f"{what}: {int((err > bar).sum())} outputs beyond the bound, worst {(err / np.maximum(mag, 1e-30)).max():.3e} of mag"
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])


TENSOR_SHAPES = [
    # B, C, C_a, H, W  (bf16 NHWC, K = 13: tensor-core kernel)
    (1, 64, 16, 16, 64),      # exactly one tile
    (2, 64, 16, 17, 65),      # one pixel more in both directions
    (1, 64, 16, 5, 7),        # smaller than the kernel
    (3, 16, 16, 41, 83),      # nothing to copy through, several images
    (1, 48, 16, 90, 200),     # several tiles per CTA in both directions
    (1, 64, 16, 1, 300),      # single row
    (1, 64, 16, 150, 1),      # single column
    (40, 32, 16, 40, 40),     # 120 tiles: one per CTA, many images
    (1, 64, 16, 360, 640),    # 230 tiles of 64x16: two per CTA on 148 SMs (the benchmark's launch)
    (1, 64, 16, 700, 130),    # tcgen05 kernel: two strips of 128 pixels (the second two pixels wide), 70 row ranges of 10 rows
    (60, 32, 16, 100, 40),    # tcgen05 kernel: row ranges of 50 rows -- the 32 row slots of tensor memory and the ring of 16 input
                              # rows are re-used inside a CTA, the issuing thread waits for the epilogue's progress
    (150, 16, 16, 70, 20),    # more images than SMs: one CTA per image, 70 rows each (two wraps of the row slots)
    (50, 32, 16, 96, 128),    # 600 tiles: four or five per CTA -- both buffers re-used, the barrier phase wraps,
                              # the image (and its dk) changes inside a CTA's walk
]


@pytest.mark.parametrize("shape", TENSOR_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("forward", [True, False], ids=["forward", "stencil"])
@pytest.mark.parametrize("engine", [0, 1], ids=["tcgen05", "mma_sync"])
def test_dense_tensor_core_kernel(pkg, oracle, shape, forward, engine):
    """Both tensor-core kernels of the dense large kernel (tcgen05 with accumulators in tensor memory, path 5;
    warp-level mma.sync, path 3) on every shape, every output compared with the oracle."""
    import torch

    B, C, C_a, H, W = shape
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape), per_image_scale=True, channel_means=True)
    wd = synth.make_dense_kernel(C_a, K, synth.BF16, seed=sum(shape))
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    _, wdyn, bdyn = util.weights_to_device(d, synth.BF16)
    wd_d = torch.from_numpy(wd).to("cuda", torch.bfloat16)
    n = x.numel()
    buf = torch.full((n + 2048,), 7.0, dtype=x.dtype, device="cuda")
    out = buf[1024:1024 + n].view(x.shape)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_set_dense_engine(engine)
    try:
        for _ in range(2):                                 # twice: barriers, rings and tensor memory start clean each launch
            if forward:
                pkg.esc_convattn_forward_dense(x, C_a, K, wd_d, wdyn, bdyn, out, pkg.ESC_NHWC, ws)
            else:
                dk = np.random.default_rng(7).uniform(-0.5, 0.5, size=(B, C_a, 3, 3)).astype(np.float32)
                pkg.esc_convattn_stencil_dense(x, C_a, K, wd_d, torch.from_numpy(dk).cuda(), out, pkg.ESC_NHWC, ws)
        torch.cuda.synchronize()
    finally:
        pkg.esc_convattn_set_dense_engine(0)
    assert pkg.esc_convattn_device_status(ws) == 0
    assert pkg.esc_convattn_last_path() == (5 if engine == 0 else 3)
    assert bool((buf[:1024] == 7.0).all()) and bool((buf[1024 + n:] == 7.0).all()), "write outside out"
    if forward:
        ref, mag = oracle.forward_dense(d["x"], C_a, wd, d["w_dyn"], d["b_dyn"], want_mag=True)
    else:
        ref, mag = oracle.stencil_dense(d["x"], C_a, wd, dk, want_mag=True)
    _check(util.to_host_nchw(out, synth.NHWC), ref, mag, synth.BF16, C_a, f"dense {shape}")


GENERIC_SHAPES = [
    # B, C, C_a, H, W, K
    (2, 24, 16, 19, 23, 13),
    (1, 20, 12, 15, 17, 5),
    (1, 40, 32, 9, 30, 13),      # C_a = 32 also for bf16 NHWC: not the tensor-core kernel's shape
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", GENERIC_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_dense_every_type_and_layout(pkg, oracle, shape, dtype, layout):
    import torch

    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), channel_means=True)
    wd = synth.make_dense_kernel(C_a, K, dtype, seed=sum(shape))
    x = util.to_device(d["x"], dtype, layout)
    _, wdyn, bdyn = util.weights_to_device(d, dtype)
    out = torch.full_like(x, 7.0)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_forward_dense(x, C_a, K, torch.from_numpy(wd).to("cuda", util.torch_dtype(dtype)), wdyn, bdyn, out,
                                   util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    fast = dtype == synth.BF16 and layout == synth.NHWC and K == 13 and C_a == 16
    assert pkg.esc_convattn_last_path() == (5 if fast else 1)
    ref, mag = oracle.forward_dense(d["x"], C_a, wd, d["w_dyn"], d["b_dyn"], want_mag=True)
    _check(util.to_host_nchw(out, layout), ref, mag, dtype, C_a, f"dense {shape} {dtype} {layout}")


def test_diagonal_dense_kernel_matches_the_depthwise_path(pkg):
    """A dense kernel that is diagonal in (output, input) channel is the depth-wise module: the tensor-core
    kernel and the register-tiled kernel must agree to fp32 summation order (both round once to bf16)."""
    import torch

    B, C, C_a, H, W, K = 1, 64, 16, 70, 100, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=31, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, wdyn, bdyn = util.weights_to_device(d, synth.BF16)
    wd = torch.zeros(C_a, C_a, K, K, dtype=torch.bfloat16, device="cuda")
    for c in range(C_a):
        wd[c, c] = wl[c]
    ws = pkg.new_workspace(B, C_a, H, W, K)
    a, b = torch.empty_like(x), torch.empty_like(x)
    pkg.esc_convattn_forward_ex(x, C_a, K, wl, wdyn, bdyn, a, pkg.ESC_NHWC, ws)
    pkg.esc_convattn_forward_dense(x, C_a, K, wd, wdyn, bdyn, b, pkg.ESC_NHWC, ws)
    torch.cuda.synchronize()
    af, bf = a.float(), b.float()
    assert torch.equal(a[..., C_a:].contiguous().view(torch.int16), b[..., C_a:].contiguous().view(torch.int16))
    diff = (af - bf).abs()[..., :C_a]
    assert bool((diff <= 2.0 ** -7 * af[..., :C_a].abs() + 1e-3).all())      # at most one bf16 ulp apart
    assert float((diff > 0).float().mean()) < 0.05                           # and nearly always identical
