"""GPU parity for the two-layer kernel estimator (ESC paper, Section 3.3, Eq. 4 line 2 as written:
two 1x1 convolutions on the pooled vector with the exact Gaussian error linear unit between them),
through the C ABI against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

LAYOUTS = [synth.NCHW, synth.NHWC]
DTYPES = [synth.F32, synth.BF16]
MLP_KEYS = ("w_down", "b_down", "w_up", "b_up")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


def mlp_to_device(m, dtype):
    import torch

    return tuple(torch.from_numpy(m[k]).to("cuda", util.torch_dtype(dtype)) for k in MLP_KEYS)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("h", [1, 4, 8, 24, 128])
def test_dk_stage_mlp(pkg, oracle, h, dtype, layout):
    """GAP + two-layer estimator on non-zero-mean data: dk within 1e-5 of max|dk| (fp32 arithmetic)."""
    import torch

    for (B, C, C_a, H, W) in [(3, 64, 16, 37, 53), (1, 192, 48, 40, 60), (2, 24, 8, 16, 16), (70, 32, 16, 8, 8)]:
        d = synth.make_inputs(B, C, C_a, H, W, 13, dtype, seed=B * 100 + H + h, channel_means=True)
        m = synth.make_estimator_mlp(C_a, h, dtype, seed=h + B)
        x = util.to_device(d["x"], dtype, layout)
        dev = mlp_to_device(m, dtype)
        dk = torch.full((B, C_a, 3, 3), float("nan"), device="cuda")
        ws = pkg.new_workspace(B, C_a, H, W, 13)
        for _ in range(2):  # twice: the arrival counters must be ready for reuse
            pkg.esc_convattn_dynkernel_mlp(x, C_a, *dev, dk, util.layout_code(layout), ws)
        torch.cuda.synchronize()
        ref, hid = oracle.dynkernel_mlp(oracle.gap(d["x"], C_a), *(m[k] for k in MLP_KEYS), want_hidden=True)
        # the inputs must exercise the curved part of the activation, not only its linear tails
        if h >= 4:
            pre = oracle.gap(d["x"], C_a) @ m["w_down"].astype(np.float64).T + m["b_down"]
            assert (np.abs(pre) < 1.5).any() and (pre < -0.5).any() and (pre > 0.5).any()
        err = np.abs(dk.cpu().numpy().astype(np.float64) - ref).max()
        assert err <= 1e-5 * max(np.abs(ref).max(), np.abs(hid).max()), (B, C, C_a, H, W, h, err)


FORWARD_SHAPES = [
    # B, C, C_a, H, W, K, h
    (2, 64, 16, 64, 64, 13, 8),     # training patches, ESC / ESC-light estimator width
    (1, 48, 16, 45, 77, 13, 4),     # ESC-FP: C = 48, h = 4
    (1, 192, 48, 50, 70, 13, 24),   # the larger model: C = 192, 48 attention channels, h = 24
    (1, 64, 16, 90, 130, 13, 8),
    (1, 20, 12, 19, 23, 3, 5),      # generic path, odd sizes
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", FORWARD_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_mlp(pkg, oracle, shape, dtype, layout):
    import torch

    B, C, C_a, H, W, K, h = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), per_image_scale=True, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, dtype, seed=sum(shape))
    x = util.to_device(d["x"], dtype, layout)
    wl = torch.from_numpy(d["w_large"]).to("cuda", util.torch_dtype(dtype))
    dev = mlp_to_device(m, dtype)
    out = torch.full_like(x, 7.0)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_forward_mlp(x, C_a, K, wl, *dev, out, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    ref, mag = oracle.forward_mlp(d["x"], C_a, d["w_large"], *(m[k] for k in MLP_KEYS), want_mag=True)
    got = util.to_host_nchw(out, layout)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, dtype, f"mlp {shape}")
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])
    if dtype == synth.BF16 and layout == synth.NHWC and K == 13:
        assert pkg.esc_convattn_last_path() in (2, 4)


def test_mlp_differs_from_linear_and_rejects_bad_width(pkg, oracle):
    """The activation is really applied (the result is not the composed linear map), and hidden widths
    outside 1..128 are refused before anything is enqueued."""
    import torch

    B, C, C_a, H, W, h = 1, 32, 16, 20, 20, 8
    d = synth.make_inputs(B, C, C_a, H, W, 13, synth.F32, seed=77, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, synth.F32, seed=77)
    x = util.to_device(d["x"], synth.F32, synth.NCHW)
    dev = mlp_to_device(m, synth.F32)
    dk = torch.zeros(B, C_a, 3, 3, device="cuda")
    ws = pkg.new_workspace(B, C_a, H, W, 13)
    pkg.esc_convattn_dynkernel_mlp(x, C_a, *dev, dk, pkg.ESC_NCHW, ws)
    torch.cuda.synchronize()
    wd, bd, wu, bu = (m[k].astype(np.float64) for k in MLP_KEYS)
    composed = oracle.dynkernel(oracle.gap(d["x"], C_a), wu @ wd, wu @ bd + bu)
    assert np.abs(dk.cpu().numpy() - composed).max() > 1e-2
    L = pkg.lib()
    args = lambda hidden: (x.data_ptr(), B, C, C_a, H, W, dev[0].data_ptr(), dev[1].data_ptr(), dev[2].data_ptr(),
                           dev[3].data_ptr(), hidden, dk.data_ptr(), pkg.ESC_F32, pkg.ESC_NCHW, ws.data_ptr(),
                           ws.numel(), None)
    for bad in (0, -1, 129):
        assert L.esc_convattn_dynkernel_mlp(*args(bad)) == 2   # ESC_ERR_SHAPE
