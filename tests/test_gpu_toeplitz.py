"""GPU parity of the tensor-core (banded Toeplitz) form of the depth-wise stage (ESC paper, Section 3.3,
Eq. 4 line 3 with the large kernel of Eq. 5's depth-wise form) against the CPU oracle, every output
compared.  Bar: one bf16 rounding of the result plus fp32 accumulation noise (tests/util.py)."""
import contextlib

import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util
from tests.test_gpu_parity import TILE_SHAPES, compare_full

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


@contextlib.contextmanager
def engine(pkg, which):
    pkg.esc_convattn_set_stencil_engine(which)
    try:
        yield
    finally:
        pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)


@pytest.mark.parametrize("shape", TILE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_tensor_engine(pkg, oracle, shape):
    """Every shape the kernel accepts: maps smaller than the kernel, single rows and columns, ragged tails,
    one to three channel groups, no and many copy-through channels."""
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + 4, per_image_scale=True, channel_means=True)
    with engine(pkg, pkg.ESC_ENGINE_TENSOR):
        compare_full(pkg, oracle, d, C_a, K, synth.BF16, synth.NHWC, what=f"{shape} tensor engine")
        assert pkg.esc_convattn_last_path() == 4


def test_engines_agree_and_switch(pkg, oracle):
    """The same call on either engine: both within the bar of the oracle, the switch selects the kernel, an
    unknown engine is refused and leaves the choice alone."""
    B, C, C_a, H, W, K = 2, 64, 16, 77, 150, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=31, per_image_scale=True, channel_means=True)
    for which, path in ((pkg.ESC_ENGINE_FP32, 2), (pkg.ESC_ENGINE_TENSOR, 4), (pkg.ESC_ENGINE_AUTO, 4)):
        with engine(pkg, which):
            compare_full(pkg, oracle, d, C_a, K, synth.BF16, synth.NHWC, what=f"engine {which}")
            assert pkg.esc_convattn_last_path() == path
    with pytest.raises(pkg.EscError):
        pkg.esc_convattn_set_stencil_engine(7)
    # shapes the tensor-core kernel does not take fall to the guarded generic kernel when it is demanded
    d = synth.make_inputs(1, 20, 12, 19, 23, 13, synth.BF16, seed=32, channel_means=True)
    with engine(pkg, pkg.ESC_ENGINE_TENSOR):
        compare_full(pkg, oracle, d, 12, 13, synth.BF16, synth.NHWC, what="C_a = 12")
        assert pkg.esc_convattn_last_path() == 1


def test_many_units_per_cta(pkg, oracle):
    """Eight images, two channel groups, 280x400: 2,016 units of 64x16, thirteen or fourteen per CTA on 148
    SMs, with image and channel-group changes inside every CTA's walk; all outputs compared."""
    B, C, C_a, H, W, K = 8, 64, 32, 280, 400, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=2031, per_image_scale=True, channel_means=True)
    with engine(pkg, pkg.ESC_ENGINE_TENSOR):
        compare_full(pkg, oracle, d, C_a, K, synth.BF16, synth.NHWC, what="many units, tensor engine")
        assert pkg.esc_convattn_last_path() == 4


def test_stencil_stage_explicit_dk_and_determinism(pkg, oracle):
    """The stage alone with a given dk (so that a wrong 3x3 tap order cannot hide behind small dynamic taps),
    and bitwise identical results run to run."""
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 45, 70, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=78)
    dk = np.random.default_rng(6).uniform(-0.5, 0.5, size=(B, C_a, 3, 3)).astype(np.float32)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, _, _ = util.weights_to_device(d, synth.BF16)
    outs = []
    with engine(pkg, pkg.ESC_ENGINE_TENSOR):
        for _ in range(3):
            out = torch.empty_like(x)
            pkg.esc_convattn_stencil(x, C_a, K, wl, torch.from_numpy(dk).cuda(), out, pkg.ESC_NHWC)
            torch.cuda.synchronize()
            assert pkg.esc_convattn_last_path() == 4
            outs.append(out)
    ref, mag = oracle.stencil(d["x"], C_a, d["w_large"], dk, want_mag=True)
    got = util.to_host_nchw(outs[0], synth.NHWC)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, "stencil stage, tensor engine", unit_variance=True)
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16)) and torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))


@pytest.mark.parametrize("shape", [(1, 64, 16, 300, 640), (70, 32, 16, 40, 64), (16, 64, 32, 33, 70), (14, 48, 48, 30, 90), (1, 64, 16, 100, 150),
                                   (1, 64, 16, 540, 960), (100, 32, 16, 64, 64), (3, 64, 32, 200, 400), (1, 48, 16, 700, 1000)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("mode", ["one_launch", "unaligned", "two_launches"])
def test_one_launch_forward_estimator_inputs(pkg, oracle, shape, mode):
    """The one-launch forward (stage 1 inside the stencil kernel; a CTA evaluates the estimator for both of its
    units at once), the same with the estimator's weights at an address that is only 2-byte aligned, and
    "two_launches": the same forward with stage 1 as its own kernel.
    Shapes: one image with two units per CTA (190 units), 210 / 192 / 168 units whose image and channel group change
    between a CTA's two units (one, two, three groups), a launch with fewer units than SMs, and 510 / 400 / 546 / 704
    units: CTAs walk three to five units, whose interiors pass through the two half-tile slots before the first products.  All outputs compared with the oracle, twice (the counters and flags are re-used)."""
    import torch

    B, C, C_a, H, W = shape
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + 9, per_image_scale=True, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    if mode == "unaligned":
        hold_w = torch.empty(wd.numel() + 8, dtype=wd.dtype, device="cuda")
        hold_b = torch.empty(bd.numel() + 8, dtype=bd.dtype, device="cuda")
        hold_w[1:1 + wd.numel()] = wd.reshape(-1)
        hold_b[1:1 + bd.numel()] = bd.reshape(-1)
        wd, bd = hold_w[1:1 + wd.numel()].view(wd.shape), hold_b[1:1 + bd.numel()].view(bd.shape)
        assert wd.data_ptr() % 16 == 2
    ws = pkg.new_workspace(B, C_a, H, W, K)
    out = torch.full_like(x, 7.0)
    pkg.esc_convattn_set_fused_stage1(mode != "two_launches")
    try:
        for _ in range(2):
            pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, pkg.ESC_NHWC, ws)
        torch.cuda.synchronize()
    finally:
        pkg.esc_convattn_set_fused_stage1(True)
    assert pkg.esc_convattn_device_status(ws) == 0
    assert pkg.esc_convattn_last_path() == 4
    assert pkg.esc_convattn_last_launches() == (2 if mode == "two_launches" else 1)
    ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
    got = util.to_host_nchw(out, synth.NHWC)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, f"{shape} {mode}")
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])


@pytest.mark.parametrize("layout", [synth.NHWC, synth.NCHW])
@pytest.mark.parametrize("shape", [(2, 64, 16, 45, 72, 9), (1, 48, 32, 70, 136, 5), (1, 64, 16, 300, 640, 11), (3, 32, 16, 20, 24, 3)],
                         ids=lambda s: "x".join(map(str, s)))
def test_smaller_large_kernels_on_the_tensor_cores(pkg, oracle, shape, layout):
    """K = 3 .. 11 (the paper's ablation of the large kernel's size): the K x K kernel is the middle of the 13 x 13 taps
    the tensor-core kernels apply, the rest zero; every output compared with the oracle run at the true K."""
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + 2, per_image_scale=True, channel_means=True)
    compare_full(pkg, oracle, d, C_a, K, synth.BF16, layout, what=f"{shape} {layout}")
    assert pkg.esc_convattn_last_path() == (4 if layout == synth.NHWC else 6)
