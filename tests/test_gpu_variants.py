"""GPU parity for the module as the paper's model variants use it (ESC paper, Sections 3.2 and 3.3): ESC and
ESC-light -- dense large kernel with the two-layer estimator; ESC-FP -- decomposed large kernel (Eq. 5) with the
two-layer estimator; through esc_convattn_forward_variant against the CPU oracle."""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
MLP_KEYS = ("w_down", "b_down", "w_up", "b_up")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


VARIANTS = [
    # name, large kernel, C, hidden, H, W
    ("ESC: dense LK, h=8", "dense", 64, 8, 40, 90),
    ("ESC-FP: decomposed LK, h=4", "decomposed", 48, 4, 70, 100),
    ("ESC-FP: decomposed LK, h=8", "decomposed", 48, 8, 33, 64),
    ("depth-wise LK, h=8", "depthwise", 64, 8, 50, 80),
]


@pytest.mark.parametrize("dtype,layout", [(synth.BF16, synth.NHWC), (synth.F32, synth.NCHW)])
@pytest.mark.parametrize("variant", VARIANTS, ids=lambda v: v[0])
def test_model_variants(pkg, oracle, variant, dtype, layout):
    import torch

    _, kind, C, h, H, W = variant
    B, C_a, K = 2, 16, 13
    seed = C + h + H
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=seed, per_image_scale=True, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, dtype, seed=seed)
    tdt = util.torch_dtype(dtype)
    dev = lambda a: torch.from_numpy(a).to("cuda", tdt)
    x = util.to_device(d["x"], dtype, layout)
    out = torch.full_like(x, 7.0)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    dk = oracle.dynkernel_mlp(oracle.gap(d["x"], C_a), *(m[k] for k in MLP_KEYS))
    if kind == "dense":
        wl = synth.make_dense_kernel(C_a, K, dtype, seed=seed)
        code, wp = pkg.ESC_LK_DENSE, None
        ref, mag = oracle.stencil_dense(d["x"], C_a, wl, dk, want_mag=True)
    elif kind == "decomposed":
        wl, wp = d["w_large"], synth.make_pointwise(C_a, dtype, seed=seed)
        code = pkg.ESC_LK_DECOMPOSED
        ref, mag = oracle.stencil_pw(d["x"], C_a, wl, wp, dk, want_mag=True)
    else:
        wl, wp, code = d["w_large"], None, pkg.ESC_LK_DEPTHWISE
        ref, mag = oracle.stencil(d["x"], C_a, wl, dk, want_mag=True)
    pkg.esc_convattn_forward_variant(x, C_a, K, code, dev(wl), None if wp is None else dev(wp),
                                     *(dev(m[k]) for k in MLP_KEYS), out, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    got = util.to_host_nchw(out, layout)
    err = np.abs(got[:, :C_a] - ref[:, :C_a])
    if dtype == synth.F32:
        bar = 1e-5 * mag + 1e-30
    else:
        fast_pw = kind == "decomposed" and pkg.esc_convattn_last_path() in (2, 4)
        bar = 2.0 ** -8 * np.abs(ref[:, :C_a]) * 1.001 + (2.0 ** -8 * mag if fast_pw else 0.0) \
            + (5e-5 if kind == "dense" else 1e-5) * mag + 1e-30
        assert pkg.esc_convattn_last_path() == (5 if kind == "dense" else 4)   # decomposed: the mix runs inside the tensor-core kernel
    assert (err <= bar).all(), f"{variant[0]}: {int((err > bar).sum())} outputs beyond the bound"
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])


def test_variant_with_one_layer_estimator_is_the_plain_forward(pkg):
    import torch

    B, C, C_a, H, W, K = 1, 64, 16, 60, 90, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=5, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    a, b = torch.empty_like(x), torch.empty_like(x)
    pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, a, pkg.ESC_NHWC, ws)
    pkg.esc_convattn_forward_variant(x, C_a, K, pkg.ESC_LK_DEPTHWISE, wl, None, None, None, wd, bd, b, pkg.ESC_NHWC, ws)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    L = pkg.lib()
    assert L.esc_convattn_forward_variant(x.data_ptr(), B, C, C_a, H, W, K, 7, wl.data_ptr(), None, None, None, wd.data_ptr(),
                                          bd.data_ptr(), 0, b.data_ptr(), 1, 1, ws.data_ptr(), ws.numel(), None) == 3
