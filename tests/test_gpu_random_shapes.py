"""Seeded random sweep over shapes, element types, layouts and variants: every case is compared with the
CPU oracle like the fixed cases (ESC paper, Section 3.3, Eq. 4 / Eq. 5).  The shapes are drawn so that tile
edges, channel groups, copy-box widths and both tile geometries of the fast kernel all occur."""
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


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        C_a = int(rng.choice([8, 16, 16, 16, 32, 48]))
        C = C_a + 8 * int(rng.integers(0, 9))
        H = int(rng.choice([rng.integers(1, 20), rng.integers(20, 140)]))
        W = int(rng.choice([rng.integers(1, 20), rng.integers(20, 170)]))
        B = int(rng.integers(1, 4))
        K = int(rng.choice([13, 13, 13, 13, 5, 17]))
        dtype = synth.BF16 if rng.random() < 0.6 else synth.F32
        layout = synth.NHWC if rng.random() < 0.6 else synth.NCHW
        variant = ["plain", "mlp", "pw", "dense"][i % 4]
        if variant == "dense":                              # the oracle does 16 x K x K terms per output: keep it small
            H, W, C_a = min(H, 48), min(W, 80), 16 if rng.random() < 0.7 else C_a
            C = max(C, C_a)
        width = int(rng.choice([0, 0, 40, 64]))
        out.append((B, C, C_a, H, W, K, dtype, layout, variant, width))
    return out


CASES = _cases(60, seed=20250306)


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(map(str, c)))
def test_random_case(pkg, oracle, case):
    import torch

    B, C, C_a, H, W, K, dtype, layout, variant, width = case
    seed = abs(hash(case[:6])) % 100000
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=seed, per_image_scale=True, channel_means=True)
    tdt = util.torch_dtype(dtype)
    x = util.to_device(d["x"], dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    n = x.numel()
    buf = torch.full((n + 2048,), 7.0, dtype=x.dtype, device="cuda")      # guard bands around out
    out = buf[1024:1024 + n].view(x.shape)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    lay = util.layout_code(layout)
    pkg.esc_convattn_set_tile_width(width)
    try:
        if variant == "plain":
            pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, lay, ws)
            ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
        elif variant == "mlp":
            h = [4, 8, 24][seed % 3]
            m = synth.make_estimator_mlp(C_a, h, dtype, seed=seed)
            keys = ("w_down", "b_down", "w_up", "b_up")
            pkg.esc_convattn_forward_mlp(x, C_a, K, wl, *(torch.from_numpy(m[k]).to("cuda", tdt) for k in keys), out, lay, ws)
            ref, mag = oracle.forward_mlp(d["x"], C_a, d["w_large"], *(m[k] for k in keys), want_mag=True)
        elif variant == "dense":
            wdn = synth.make_dense_kernel(C_a, K, dtype, seed=seed)
            pkg.esc_convattn_forward_dense(x, C_a, K, torch.from_numpy(wdn).to("cuda", tdt), wd, bd, out, lay, ws)
            ref, mag = oracle.forward_dense(d["x"], C_a, wdn, d["w_dyn"], d["b_dyn"], want_mag=True)
        else:
            wp = synth.make_pointwise(C_a, dtype, seed=seed)
            pkg.esc_convattn_forward_pw(x, C_a, K, wl, torch.from_numpy(wp).to("cuda", tdt), wd, bd, out, lay, ws)
            ref, mag = oracle.forward_pw(d["x"], C_a, d["w_large"], wp, d["w_dyn"], d["b_dyn"], want_mag=True)
        torch.cuda.synchronize()
    finally:
        pkg.esc_convattn_set_tile_width(0)
    assert pkg.esc_convattn_device_status(ws) == 0
    assert bool((buf[:1024] == 7.0).all()) and bool((buf[1024 + n:] == 7.0).all()), "write outside out"
    got = util.to_host_nchw(out, layout)
    err = np.abs(got[:, :C_a] - ref[:, :C_a])
    if dtype == synth.F32:
        assert (err <= 1e-5 * mag + 1e-30).all(), f"{case}: {(err / np.maximum(mag, 1e-30)).max():.3e} of mag"
    else:
        # one bf16 rounding of the result (half an ulp: at most 2^-8 of its magnitude) on top of fp32
        # accumulation noise; where the fast kernel also keeps the mixed features in bf16, one more rounding
        # of every input of the depth-wise stage, bounded by 2^-8 of sum |w| |mixed| <= 2^-8 * mag
        extra = 2.0 ** -8 * mag if variant == "pw" and pkg.esc_convattn_last_path() in (2, 4, 6) else 0.0
        noise = 5e-5 if variant == "dense" else 1e-5       # 16 x K x K terms through the tensor cores' fp32 adders
        bar = 2.0 ** -8 * np.abs(ref[:, :C_a]) * 1.001 + extra + noise * mag + 1e-30
        assert (err <= bar).all(), f"{case}: {int((err > bar).sum())} outputs beyond the rounding bound"
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])
