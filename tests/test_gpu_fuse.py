"""GPU parity of the whole module with its closing 1x1 convolution and the block's residual (ESC paper, Section
3.3, Eq. 4 line 4; Eq. 3 line 3) through esc_convattn_forward_fused against the CPU oracle, every output compared.

Bars.  fp32: 1e-5 of the sum of absolute terms.  bf16: one rounding of the result (2^-8 |ref|) plus fp32
accumulation noise (1e-5 of the sum of absolute terms) plus, because F_res passes through a bf16 tensor between
the two kernels as it would between two layers of a bf16 network, one rounding of F_res carried through Conv_fuse:
2^-8 sum_{c < C_a} |w_fuse[n,c]| |F_res[c]|."""
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
    # B, C, C_a, H, W, K, dtype, layout, bias, residual ("x" = the input itself)
    (2, 64, 16, 45, 70, 13, synth.BF16, synth.NHWC, True, "own"),      # fast path: two or three launches, no copy-through
    (1, 64, 16, 90, 130, 13, synth.BF16, synth.NHWC, True, "x"),
    (1, 64, 16, 33, 47, 13, synth.BF16, synth.NHWC, False, None),
    (3, 48, 16, 40, 40, 13, synth.BF16, synth.NHWC, True, "own"),      # ESC-FP width
    (1, 128, 32, 30, 50, 13, synth.BF16, synth.NHWC, True, "own"),     # two channel groups, widest fast 1x1
    (1, 32, 16, 17, 65, 13, synth.BF16, synth.NHWC, True, None),
    (1, 64, 16, 300, 500, 13, synth.BF16, synth.NHWC, True, "own"),    # many units per CTA: stage 1 as a kernel of its own
    (1, 192, 48, 20, 30, 13, synth.BF16, synth.NHWC, True, "own"),     # C beyond the fast 1x1: guarded kernel in place
    (2, 24, 8, 19, 23, 13, synth.BF16, synth.NCHW, True, "own"),
    (2, 64, 16, 45, 72, 13, synth.BF16, synth.NCHW, True, "own"),      # NCHW fast path: NCHW tensor-core stencil + NCHW 1x1 kernel
    (1, 64, 16, 90, 136, 13, synth.BF16, synth.NCHW, True, "x"),       # several tiles of 128 pixels and a ragged last one
    (1, 48, 16, 33, 48, 13, synth.BF16, synth.NCHW, False, None),
    (3, 32, 16, 40, 40, 13, synth.BF16, synth.NCHW, True, "own"),
    (1, 64, 32, 300, 504, 13, synth.BF16, synth.NCHW, True, "own"),    # two channel groups, many units per CTA
    (1, 64, 16, 1, 8, 13, synth.BF16, synth.NCHW, True, "own"),        # eight pixels
    (2, 20, 12, 15, 17, 9, synth.F32, synth.NCHW, True, "own"),
    (1, 64, 16, 40, 60, 13, synth.F32, synth.NHWC, False, "x"),
]


@pytest.mark.parametrize("case", SHAPES, ids=lambda c: "x".join(map(str, c[:6])) + f"-{c[6]}-{c[7]}")
def test_forward_fused(pkg, oracle, case):
    import torch

    B, C, C_a, H, W, K, dtype, layout, with_bias, res_kind = case
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(case[:6]), per_image_scale=True, channel_means=True)
    f = synth.make_fuse(C, dtype, seed=sum(case[:6]))
    res_np = None
    if res_kind == "own":
        res_np = synth.round_to(np.random.default_rng(C + H).normal(size=d["x"].shape).astype(np.float32), dtype)
    elif res_kind == "x":
        res_np = d["x"]
    tdt = util.torch_dtype(dtype)
    x = util.to_device(d["x"], dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    wf = torch.from_numpy(f["w_fuse"]).to("cuda", tdt)
    bf = torch.from_numpy(f["b_fuse"]).to("cuda", tdt) if with_bias else None
    res = x if res_kind == "x" else util.to_device(res_np, dtype, layout) if res_kind == "own" else None
    n = x.numel()
    buf = torch.full((n + 2048,), 7.0, dtype=x.dtype, device="cuda")
    out = buf[1024:1024 + n].view(x.shape)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    for _ in range(2):
        pkg.esc_convattn_forward_fused(x, C_a, K, wl, wd, bd, wf, bf, res, out, util.layout_code(layout), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    assert bool((buf[:1024] == 7.0).all()) and bool((buf[1024 + n:] == 7.0).all()), "write outside out"
    assert pkg.esc_convattn_last_launches() in (2, 3)      # stage 1 inside the stencil kernel or before it, then the 1x1 kernel
    ref, mag, cat = oracle.forward_fused(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], f["w_fuse"],
                                         f["b_fuse"] if with_bias else None, res_np, want_mag=True, want_cat=True)
    got = util.to_host_nchw(out, layout).astype(np.float64)
    err = np.abs(got - ref)
    if dtype == synth.F32:
        bar = 1e-5 * mag + 1e-30
    else:
        carried = np.einsum("nc,bchw->bnhw", np.abs(f["w_fuse"][:, :C_a]).astype(np.float64), np.abs(cat[:, :C_a]))
        bar = 2.0 ** -8 * np.abs(ref) * 1.001 + 2.0 ** -8 * carried + 1e-5 * mag + 1e-30
    assert (err <= bar).all(), f"{case}: {int((err > bar).sum())} of {err.size} outputs beyond the bound, worst {(err / bar).max():.2f} bars"


def test_fused_identity_is_the_forward(pkg):
    """w_fuse = I without bias and residual: the call returns what esc_convattn_forward_ex returns, bit for bit
    (every bf16 value passes the 1x1 unchanged)."""
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 50, 80, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=5, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    eye = torch.eye(C, dtype=torch.bfloat16, device="cuda")
    ws = pkg.new_workspace(B, C_a, H, W, K)
    a, b = torch.empty_like(x), torch.empty_like(x)
    pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, a, pkg.ESC_NHWC, ws)
    pkg.esc_convattn_forward_fused(x, C_a, K, wl, wd, bd, eye, None, None, b, pkg.ESC_NHWC, ws)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_fused_rejections(pkg):
    import torch

    B, C, C_a, H, W, K = 1, 64, 16, 20, 20, 13
    x = torch.zeros(B, H, W, C, dtype=torch.bfloat16, device="cuda")
    wl = torch.zeros(C_a, K, K, dtype=torch.bfloat16, device="cuda")
    wd = torch.zeros(9 * C_a, C_a, dtype=torch.bfloat16, device="cuda")
    bd = torch.zeros(9 * C_a, dtype=torch.bfloat16, device="cuda")
    wf = torch.zeros(C, C, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(x)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_forward_fused(x, C_a, K, wl, wd, bd, wf, None, out, out, pkg.ESC_NHWC, ws)      # residual overlaps out
    assert e.value.status == 5
    with pytest.raises(pkg.EscError) as e:
        pkg.esc_convattn_forward_fused(x, C_a, K, wl, wd, bd, None, None, None, out, pkg.ESC_NHWC, ws)   # no w_fuse
    assert e.value.status == 1
