"""The allocation-free stage-1 entry point, esc_convattn_dynkernel_static.

Some users of this library run where device memory cannot be allocated on the fly: a control or
rendering loop whose memory is fixed at start-up, or a host framework that owns the allocator and
forbids anything else from calling cudaMalloc.  For them the library carries its scratch inside its
own device image.  This test calls that entry point through the C ABI twice in a row on each case
(the second call must find the shared scratch in a usable state) and checks the result against the
ordinary entry point that takes a caller-allocated workspace and, so that the check does not rest on
the CUDA path alone, against the CPU oracle's GAP and estimator, both to the 1e-5 bar the dk stage
test uses.  It also checks that a problem larger than the fixed scratch is refused on the host.

The file name sorts last so that a run which stops at the first failure has already run
everything else.
"""
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


@pytest.mark.parametrize("layout", [synth.NHWC, synth.NCHW])
@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_static_scratch_matches_workspace_entry(pkg, oracle, dtype, layout):
    import torch

    for (B, C, C_a, H, W) in [(1, 64, 16, 360, 640), (5, 64, 16, 64, 64), (2, 48, 32, 33, 47), (3, 20, 12, 9, 7)]:
        d = synth.make_inputs(B, C, C_a, H, W, 13, dtype, seed=900 + B + H, channel_means=True)
        x = util.to_device(d["x"], dtype, layout)
        _, wd, bd = util.weights_to_device(d, dtype)
        ws = pkg.new_workspace(B, C_a, H, W, 13)
        ref = torch.full((B, C_a, 3, 3), float("nan"), device="cuda")
        pkg.esc_convattn_dynkernel(x, C_a, wd, bd, ref, util.layout_code(layout), ws)
        torch.cuda.synchronize()
        scale = float(ref.abs().max())
        want = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"]).reshape(B, C_a, 3, 3)
        for call in range(2):   # two calls in a row share the same fixed scratch
            got = torch.full((B, C_a, 3, 3), float("nan"), device="cuda")   # allocated by the test, not the call
            pkg.esc_convattn_dynkernel_static(x, C_a, wd, bd, got, util.layout_code(layout))
            torch.cuda.synchronize()
            err = float((got - ref).abs().max())
            assert err <= 1e-5 * scale, (dtype, layout, (B, C, C_a, H, W), call, err)
            err_o = float(np.abs(got.cpu().numpy().astype(np.float64) - want).max())
            assert err_o <= 1e-5 * np.abs(want).max(), ("against the oracle", dtype, layout, (B, C, C_a, H, W), call, err_o)


def test_static_scratch_refuses_oversized_problem(pkg):
    import torch

    B, C, C_a, H, W = 1100, 16, 16, 8, 8        # more images than the fixed scratch has arrival counters
    x = torch.zeros(B, H, W, C, device="cuda", dtype=torch.bfloat16)
    wd = torch.zeros(9 * C_a, C_a, device="cuda", dtype=torch.bfloat16)
    bd = torch.zeros(9 * C_a, device="cuda", dtype=torch.bfloat16)
    dk = torch.zeros(B, C_a, 3, 3, device="cuda")
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_dynkernel_static(x, C_a, wd, bd, dk, pkg.ESC_NHWC)
    assert e.value.status == 6 and "fixed scratch" in pkg.esc_last_error()
    B = 32                                      # 32 images x 4 slabs x 128 channels > 15360 partial sums
    x = torch.zeros(B, 128, 128, 128, device="cuda", dtype=torch.bfloat16)
    wd = torch.zeros(9 * 128, 128, device="cuda", dtype=torch.bfloat16)
    bd = torch.zeros(9 * 128, device="cuda", dtype=torch.bfloat16)
    dk = torch.zeros(B, 128, 3, 3, device="cuda")
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_dynkernel_static(x, 128, wd, bd, dk, pkg.ESC_NHWC)
    assert e.value.status == 6
