"""GPU parity of the tensor-core (banded Toeplitz) depth-wise kernel for NCHW bf16 tensors (ESC paper, Section 3.3,
Eq. 4 lines 3-4) against the CPU oracle, every output compared; identity channels bit for bit."""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


SHAPES = [
    # B, C, C_a, H, W   (W a multiple of 8: rows are whole 16-byte pieces, which the tile loads need)
    (1, 64, 16, 16, 64),      # exactly one tile
    (2, 64, 16, 17, 72),      # one row and eight columns more
    (1, 64, 16, 5, 8),        # smaller than the kernel, narrower than a tile's halo
    (3, 16, 16, 41, 88),      # nothing to copy through, several images
    (1, 48, 32, 90, 200),     # two channel groups, several tiles in both directions
    (1, 64, 16, 1, 304),      # single row
    (1, 64, 16, 150, 8),      # eight columns
    (1, 64, 16, 300, 640),    # 190 units: two per CTA on 148 SMs, one launch for the whole forward
    (70, 32, 16, 40, 64),     # 210 units: a CTA's two units belong to two images
    (16, 64, 32, 33, 72),     # 192 units: image and channel group change between a CTA's two units
    (14, 48, 48, 30, 96),     # three channel groups, nothing to copy through
    (8, 64, 32, 280, 400),    # 2,016 units: thirteen or fourteen per CTA, both buffers re-used many times, two launches
    (3, 192, 48, 70, 120),    # the larger model's channel counts: 144 identity channels
    (1, 64, 16, 540, 960),    # 510 units: three or four per CTA, two launches
    (100, 32, 16, 64, 64),    # 400 units: three per CTA, every one of another image
    (3, 64, 32, 200, 400),    # 546 units: image and channel group change inside a CTA's walk of three or four
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("one_launch", [True, False], ids=["one_launch", "two_launches"])
def test_forward_nchw(pkg, oracle, shape, one_launch):
    import torch

    B, C, C_a, H, W = shape
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + 17, per_image_scale=True, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NCHW)
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    n = x.numel()
    buf = torch.full((n + 2048,), 7.0, dtype=x.dtype, device="cuda")
    out = buf[1024:1024 + n].view(x.shape)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_set_fused_stage1(one_launch)
    try:
        for _ in range(2):                                 # twice: counters, flags and barriers start clean each launch
            pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, pkg.ESC_NCHW, ws)
        torch.cuda.synchronize()
    finally:
        pkg.esc_convattn_set_fused_stage1(True)
    assert pkg.esc_convattn_device_status(ws) == 0
    assert pkg.esc_convattn_last_path() == 6
    units = B * (C_a // 16) * ((W + 63) // 64) * ((H + 15) // 16)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert pkg.esc_convattn_last_launches() == (1 if one_launch and units <= 2 * sms else 2)
    assert bool((buf[:1024] == 7.0).all()) and bool((buf[1024 + n:] == 7.0).all()), "write outside out"
    ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
    got = util.to_host_nchw(out, synth.NCHW)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, f"nchw {shape}")
    assert torch.equal(x[:, C_a:].contiguous().view(torch.int16), out[:, C_a:].contiguous().view(torch.int16))


def test_stencil_stage_explicit_dk_nchw(pkg, oracle):
    """The stage alone with a given dk of ordinary size (a wrong 3x3 tap order or column offset cannot hide behind
    small dynamic taps), bitwise identical run to run."""
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 45, 72, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=79)
    dk = np.random.default_rng(8).uniform(-0.5, 0.5, size=(B, C_a, 3, 3)).astype(np.float32)
    x = util.to_device(d["x"], synth.BF16, synth.NCHW)
    wl, _, _ = util.weights_to_device(d, synth.BF16)
    outs = []
    for _ in range(3):
        out = torch.empty_like(x)
        pkg.esc_convattn_stencil(x, C_a, K, wl, torch.from_numpy(dk).cuda(), out, pkg.ESC_NCHW)
        torch.cuda.synchronize()
        assert pkg.esc_convattn_last_path() == 6
        outs.append(out)
    ref, mag = oracle.stencil(d["x"], C_a, d["w_large"], dk, want_mag=True)
    got = util.to_host_nchw(outs[0], synth.NCHW)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, "stencil stage, nchw tensor kernel", unit_variance=True)
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16)) and torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))


def test_shapes_the_kernel_does_not_take_fall_back(pkg, oracle):
    """Rows that are not whole 16-byte pieces (W = 70), C_a = 12, and the FP32 engine: the guarded generic kernel."""
    import torch

    for (B, C, C_a, H, W), engine in [((1, 32, 16, 20, 70), None), ((1, 20, 12, 19, 24), None), ((1, 32, 16, 20, 72), "fp32")]:
        d = synth.make_inputs(B, C, C_a, H, W, 13, synth.BF16, seed=5 + W, channel_means=True)
        x = util.to_device(d["x"], synth.BF16, synth.NCHW)
        wl, wd, bd = util.weights_to_device(d, synth.BF16)
        out = torch.empty_like(x)
        ws = pkg.new_workspace(B, C_a, H, W, 13)
        if engine:
            pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
        try:
            pkg.esc_convattn_forward_ex(x, C_a, 13, wl, wd, bd, out, pkg.ESC_NCHW, ws)
            torch.cuda.synchronize()
        finally:
            pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)
        assert pkg.esc_convattn_last_path() == 1
        ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
        got = util.to_host_nchw(out, synth.NCHW)
        util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, f"fallback {(B, C, C_a, H, W)}")
        assert np.array_equal(got[:, C_a:], ref[:, C_a:])
