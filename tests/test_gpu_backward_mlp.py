"""GPU parity of esc_convattn_backward_mlp -- the backward pass with the estimator as the paper writes it (ESC Section
3.3, Eq. 4 line 2: two layers, exact GELU) -- through the C ABI against the CPU oracle's backward_mlp."""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
KEYS = ("w_down", "b_down", "w_up", "b_up")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


CASES = [
    # B, C, C_a, H, W, hidden
    (2, 64, 16, 64, 64, 8),       # ESC / ESC-light widths
    (1, 48, 16, 70, 131, 4),      # ESC-FP width, ragged tiles
    (3, 24, 8, 9, 11, 5),         # smaller than the kernel, C_a = 8
    (1, 48, 32, 37, 90, 24),      # two channel groups, the larger model's hidden width
    (6, 32, 16, 130, 200, 8),     # 216 units of 64x16 on the tensor-core path: CTAs walk two units
]


@pytest.mark.parametrize("dtype,layout", [(synth.BF16, synth.NHWC), (synth.BF16, synth.NCHW), (synth.F32, synth.NCHW), (synth.F32, synth.NHWC)])
@pytest.mark.parametrize("case", CASES, ids=lambda s: "x".join(map(str, s)))
def test_backward_mlp(pkg, oracle, case, dtype, layout):
    import torch

    B, C, C_a, H, W, h = case
    K = 13
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(case), per_image_scale=True, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, dtype, seed=sum(case))
    go = synth.round_to(np.random.default_rng(sum(case) + 1).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    tdt = util.torch_dtype(dtype)
    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(go, dtype, layout)
    wl = torch.from_numpy(d["w_large"]).to("cuda", tdt)
    mlp = [torch.from_numpy(m[k]).to("cuda", tdt) for k in KEYS]
    gx = torch.full_like(x, 7.0)
    nan = float("nan")
    g_lk = torch.full((C_a, K, K), nan, device="cuda")
    g_wd = torch.full((h, C_a), nan, device="cuda")
    g_bd = torch.full((h,), nan, device="cuda")
    g_wu = torch.full((9 * C_a, h), nan, device="cuda")
    g_bu = torch.full((9 * C_a,), nan, device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    for _ in range(2):                                   # twice: nothing in the workspace may need re-zeroing
        pkg.esc_convattn_backward_mlp(x, go_d, C_a, K, wl, *mlp, gx, g_lk, g_wd, g_bd, g_wu, g_bu, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0

    ref = oracle.backward_mlp(d["x"], go, C_a, d["w_large"], *(m[k] for k in KEYS))
    # scales of the sums: the same gradients with every term replaced by its magnitude and phi' by its bound 1.13
    mabs = {k: np.abs(m[k]) for k in KEYS}
    gmean = np.abs(oracle.gap(np.abs(d["x"]), C_a))
    _, alk, _, ab1 = oracle.backward(np.abs(d["x"]), np.abs(go), C_a, d["w_large"], np.zeros((9 * C_a, C_a)), np.zeros(9 * C_a))
    # ab1 = sum_b |g_dk| bound per output o (from |x|, |go|); per image bound: use the same (B small) as a scale
    a_act = np.abs(gmean @ mabs["w_down"].T + mabs["b_down"])                       # |a| <= |t|
    s_bu = ab1
    s_wu = np.outer(ab1, a_act.max(axis=0))
    s_ga = ab1 @ mabs["w_up"]                                                       # [h]
    s_bd = 1.13 * s_ga
    s_wd = np.outer(s_bd, gmean.max(axis=0))
    tol = 2e-5 if dtype == synth.F32 else 2e-5
    for name, got, r, scale in (("w_large", g_lk, ref[1], alk), ("w_down", g_wd, ref[2], s_wd), ("b_down", g_bd, ref[3], s_bd),
                                ("w_up", g_wu, ref[4], s_wu), ("b_up", g_bu, ref[5], s_bu)):
        err = np.abs(got.cpu().numpy().astype(np.float64) - r)
        assert np.isfinite(got.cpu().numpy()).all(), name
        assert (err <= tol * scale + 1e-30).all(), f"grad {name}: worst {(err / np.maximum(scale, 1e-30)).max():.3e} of its scale"

    got = util.to_host_nchw(gx, layout)
    assert np.array_equal(got[:, C_a:], go[:, C_a:].astype(np.float64)), "identity channels: grad_x must be grad_out"
    dk = oracle.dynkernel_mlp(oracle.gap(d["x"], C_a), *(m[k] for k in KEYS))
    mag = oracle.stencil(np.abs(go), C_a, np.abs(d["w_large"][:, ::-1, ::-1]).copy(), np.abs(dk[:, :, ::-1, ::-1]).copy())[:, :C_a]
    err = np.abs(got[:, :C_a] - ref[0][:, :C_a])
    gg_scale = (s_bd @ mabs["w_down"]) / (H * W)                                    # [C_a]: bound of the GAP-path constant
    bar = 1e-5 * mag + 2e-5 * gg_scale[None, :, None, None] + 1e-30
    if dtype == synth.BF16:
        bar = bar + 2.0 ** -8 * np.abs(ref[0][:, :C_a]) * 1.001
    assert (err <= bar).all(), f"grad x: {int((err > bar).sum())} values beyond the bound"


def test_backward_mlp_rejections(pkg):
    import torch

    B, C, C_a, H, W, K, h = 1, 32, 16, 20, 24, 13, 8
    x = torch.zeros(B, H, W, C, dtype=torch.bfloat16, device="cuda")
    go, gx = torch.zeros_like(x), torch.zeros_like(x)
    wl = torch.zeros(C_a, K, K, dtype=torch.bfloat16, device="cuda")
    wdn, bdn = torch.zeros(h, C_a, dtype=torch.bfloat16, device="cuda"), torch.zeros(h, dtype=torch.bfloat16, device="cuda")
    wup, bup = torch.zeros(9 * C_a, h, dtype=torch.bfloat16, device="cuda"), torch.zeros(9 * C_a, dtype=torch.bfloat16, device="cuda")
    ws = pkg.new_backward_workspace(B, C_a, H, W, K)
    with pytest.raises(pkg.EscError):                       # grad_x must not overlap x
        pkg.esc_convattn_backward_mlp(x, go, C_a, K, wl, wdn, bdn, wup, bup, x, None, None, None, None, None, pkg.ESC_NHWC, ws)
    big = torch.zeros(200, C_a, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pkg.EscError):                       # hidden beyond the limit
        pkg.esc_convattn_backward_mlp(x, go, C_a, K, wl, big, torch.zeros(200, dtype=torch.bfloat16, device="cuda"),
                                      torch.zeros(9 * C_a, 200, dtype=torch.bfloat16, device="cuda"), bup, gx, None, None, None, None, None,
                                      pkg.ESC_NHWC, ws)
    # all weight gradients may be left out
    pkg.esc_convattn_backward_mlp(x, go, C_a, K, wl, wdn, bdn, wup, bup, gx, None, None, None, None, None, pkg.ESC_NHWC, ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
