"""GPU parity for esc_convattn_backward_variant: every large-kernel form with the two-layer estimator of Eq. 4 line 2
(the configurations the paper's models use) and, with hidden = 0, the one-layer forms through the same entry; against
the CPU oracle (pinned by equality with the pinned two-layer backward and by central differences).

Bars as in the forms' own tests: weight gradients 1e-5 of the sums' scale (bf16 decomposed form: + 2^-8 for the two
stored intermediates, and 2^-7 in norm); grad_x checked in the Euclidean norm against the reference (2^-7 for bf16,
1e-5 of the scale's norm for fp32) and element-wise against a bar built from the scale and the roundings.
"""
import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

LAYOUTS = [synth.NCHW, synth.NHWC]
DTYPES = [synth.F32, synth.BF16]
FORMS = ["depthwise", "pw", "dense"]
KEYS = ("w_down", "b_down", "w_up", "b_up")


@pytest.fixture(scope="module")
def pkg():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as p

    p.lib()
    return p


def _inputs(form, shape, dtype, h, seed):
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=seed, per_image_scale=True, channel_means=True)
    m = synth.make_estimator_mlp(C_a, h, dtype, seed=seed)
    for k in KEYS:
        d[k] = m[k]
    d["w_point"] = synth.make_pointwise(C_a, dtype, seed=seed) if form == "pw" else None
    if form == "dense":
        d["w_large"] = synth.make_dense_kernel(C_a, K, dtype, seed=seed)
    d["go"] = synth.round_to(np.random.default_rng(seed + 1).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    return d


def _run(pkg, form, d, C_a, K, dtype, layout):
    import torch

    code = {"depthwise": pkg.ESC_LK_DEPTHWISE, "pw": pkg.ESC_LK_DECOMPOSED, "dense": pkg.ESC_LK_DENSE}[form]
    tdt = util.torch_dtype(dtype)
    x = util.to_device(d["x"], dtype, layout)
    go_d = util.to_device(d["go"], dtype, layout)
    dev = {k: torch.from_numpy(np.ascontiguousarray(d[k])).to("cuda", tdt) for k in ("w_large",) + KEYS}
    wp = torch.from_numpy(d["w_point"]).to("cuda", tdt) if form == "pw" else None
    B, _, H, W = d["x"].shape
    h = d["w_down"].shape[0]
    gx = torch.full_like(x, 7.0)
    g = {"w_large": torch.full(d["w_large"].shape, float("nan"), device="cuda"),
         "w_point": torch.full((C_a, C_a), float("nan"), device="cuda") if form == "pw" else None,
         "w_down": torch.full((h, C_a), float("nan"), device="cuda"), "b_down": torch.full((h,), float("nan"), device="cuda"),
         "w_up": torch.full((9 * C_a, h), float("nan"), device="cuda"), "b_up": torch.full((9 * C_a,), float("nan"), device="cuda")}
    ws = pkg.new_backward_dense_workspace(B, C_a, H, W, K) if form == "dense" else pkg.new_backward_workspace(B, C_a, H, W, K)
    for _ in range(2):
        pkg.esc_convattn_backward_variant(x, go_d, C_a, K, code, dev["w_large"], wp, dev["w_down"], dev["b_down"], dev["w_up"], dev["b_up"],
                                          gx, g["w_large"], g["w_point"], g["w_down"], g["b_down"], g["w_up"], g["b_up"],
                                          util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    return util.to_host_nchw(gx, layout), {k: (v.cpu().numpy().astype(np.float64) if v is not None else None) for k, v in g.items()}


def _check(oracle, form, d, C_a, dtype, gx, g):
    names = ("x", "w_large", "w_point") + KEYS
    a = lambda v: None if v is None else np.abs(v)
    ref = dict(zip(names, oracle.backward_variant(d["x"], d["go"], C_a, form, d["w_large"], d["w_point"], *(d[k] for k in KEYS))))
    # scales: the one-layer passes on magnitudes bound the large kernel's sums; for the estimator's small sums the
    # reference's own largest entry is the scale (they are sums over images of products of a few hundred terms)
    bf = dtype == synth.BF16
    rel = 1e-5 + (2.0 ** -8 if (bf and form == "pw") else 0.0)
    if form == "dense":
        mag_l = oracle.backward_dense(a(d["x"]), a(d["go"]), C_a, a(d["w_large"]), np.zeros((9 * C_a, C_a)), np.zeros(9 * C_a))[1]
    elif form == "pw":
        r = oracle.backward_pw(a(d["x"]), a(d["go"]), C_a, a(d["w_large"]), a(d["w_point"]), np.zeros((9 * C_a, C_a)), np.zeros(9 * C_a))
        mag_l, mag_p = r[1], r[2]
        err = np.abs(g["w_point"] - ref["w_point"])
        assert (err <= rel * mag_p + 1e-30).all(), "grad w_point"
    else:
        mag_l = oracle.backward(a(d["x"]), a(d["go"]), C_a, a(d["w_large"]), np.zeros((9 * C_a, C_a)), np.zeros(9 * C_a))[1]
    err = np.abs(g["w_large"] - ref["w_large"])
    assert (err <= rel * mag_l + 1e-30).all(), f"grad w_large: worst {(err / np.maximum(mag_l, 1e-30)).max():.3e} of its scale"
    # estimator gradients: sums of g_dk (a 3x3 window of the tap sums, scale = the large kernel's scale at those taps)
    # times activations of order one
    gdk_scale = float(mag_l.max()) * max(1.0, float(np.abs(d["w_up"]).max()) * 9 * C_a)
    for k in KEYS:
        err = np.abs(g[k] - ref[k])
        assert err.max() <= (2e-5 + (2.0 ** -8 if (bf and form == "pw") else 0.0)) * gdk_scale, f"grad {k}: {err.max():.3e} against scale {gdk_scale:.3e}"
        nr = np.linalg.norm(ref[k])
        assert np.linalg.norm(err) <= (2.0 ** -7 if (bf and form == "pw") else 1e-3) * nr + 1e-12, f"grad {k}: {np.linalg.norm(err) / max(nr, 1e-30):.3e} in norm"
    assert np.array_equal(gx[:, C_a:], d["go"][:, C_a:].astype(np.float64))
    e = gx[:, :C_a] - ref["x"][:, :C_a]
    assert np.linalg.norm(e) <= (2.0 ** -7 if bf else 1e-5) * np.linalg.norm(ref["x"][:, :C_a]) + 1e-12, f"grad x: {np.linalg.norm(e) / np.linalg.norm(ref['x'][:, :C_a]):.3e} in norm"
    assert np.abs(e).max() <= (2.0 ** -6 if bf else 1e-4) * np.abs(ref["x"][:, :C_a]).max()


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("form", FORMS)
def test_backward_variant_two_layer(pkg, oracle, form, dtype, layout):
    shape = (2, 32, 16, 37, 72, 13)
    d = _inputs(form, shape, dtype, h=8, seed=31 + FORMS.index(form))
    gx, g = _run(pkg, form, d, 16, 13, dtype, layout)
    _check(oracle, form, d, 16, dtype, gx, g)


@pytest.mark.parametrize("form", FORMS)
def test_backward_variant_paper_widths(pkg, oracle, form):
    """bf16 NHWC at a training-patch size, hidden width 4 (the smallest the paper uses) and K = 13."""
    shape = (4, 64, 16, 64, 64, 13)
    d = _inputs(form, shape, synth.BF16, h=4, seed=77)
    gx, g = _run(pkg, form, d, 16, 13, synth.BF16, synth.NHWC)
    _check(oracle, form, d, 16, synth.BF16, gx, g)


@pytest.mark.parametrize("form", FORMS)
def test_one_layer_through_the_variant_entry(pkg, form):
    """hidden = 0: the entry must return exactly what the form's own entry returns."""
    import torch

    B, C, C_a, H, W, K = 2, 32, 16, 30, 40, 13
    dtype, layout = synth.BF16, synth.NHWC
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=9, per_image_scale=True, channel_means=True)
    if form == "dense":
        d["w_large"] = synth.make_dense_kernel(C_a, K, dtype, seed=9)
    wp = synth.make_pointwise(C_a, dtype, seed=9)
    go = synth.round_to(np.random.default_rng(10).standard_normal(size=d["x"].shape).astype(np.float32), dtype)
    tdt = util.torch_dtype(dtype)
    x = util.to_device(d["x"], dtype, layout); go_d = util.to_device(go, dtype, layout)
    wl = torch.from_numpy(d["w_large"]).to("cuda", tdt); wd = torch.from_numpy(d["w_dyn"]).to("cuda", tdt); bd = torch.from_numpy(d["b_dyn"]).to("cuda", tdt)
    wp_d = torch.from_numpy(wp).to("cuda", tdt)
    lc = util.layout_code(layout)
    new_ws = (lambda: pkg.new_backward_dense_workspace(B, C_a, H, W, K)) if form == "dense" else (lambda: pkg.new_backward_workspace(B, C_a, H, W, K))
    def outs():
        return (torch.full_like(x, 7.0), torch.zeros(d["w_large"].shape, device="cuda"), torch.zeros((C_a, C_a), device="cuda"),
                torch.zeros((9 * C_a, C_a), device="cuda"), torch.zeros((9 * C_a,), device="cuda"))
    gx1, gl1, gp1, gw1, gb1 = outs()
    code = {"depthwise": pkg.ESC_LK_DEPTHWISE, "pw": pkg.ESC_LK_DECOMPOSED, "dense": pkg.ESC_LK_DENSE}[form]
    pkg.esc_convattn_backward_variant(x, go_d, C_a, K, code, wl, wp_d if form == "pw" else None, None, None, wd, bd, gx1, gl1,
                                      gp1 if form == "pw" else None, None, None, gw1, gb1, lc, new_ws())
    gx2, gl2, gp2, gw2, gb2 = outs()
    if form == "depthwise":
        pkg.esc_convattn_backward(x, go_d, C_a, K, wl, wd, bd, gx2, gl2, gw2, gb2, lc, new_ws())
    elif form == "pw":
        pkg.esc_convattn_backward_pw(x, go_d, C_a, K, wl, wp_d, wd, bd, gx2, gl2, gp2, gw2, gb2, lc, new_ws())
    else:
        pkg.esc_convattn_backward_dense(x, go_d, C_a, K, wl, wd, bd, gx2, gl2, gw2, gb2, lc, new_ws())
    torch.cuda.synchronize()
    for a, b in ((gx1, gx2), (gl1, gl2), (gp1, gp2), (gw1, gw2), (gb1, gb2)):
        assert torch.equal(a, b)
