"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same
seeded inputs (ESC paper, Section 3.3, Eq. 4).  Tolerances are in tests/util.py."""
import contextlib

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


@contextlib.contextmanager
def tile_width(pkg, width):
    """Pins the tile geometry of the TMA-staged kernel for the calls inside (0 = chosen by cost)."""
    pkg.esc_convattn_set_tile_width(width)
    try:
        yield
    finally:
        pkg.esc_convattn_set_tile_width(0)


def run_forward(pkg, d, C_a, K, dtype, layout, entry="ex"):
    import torch

    x = util.to_device(d["x"], dtype, layout)
    wl, wd, bd = util.weights_to_device(d, dtype)
    B, C, H, W = d["x"].shape
    # guard bands around out: the kernels must not write outside it
    n = x.numel()
    pad = 4096
    buf = torch.full((n + 2 * pad,), 7.0, dtype=x.dtype, device="cuda")
    out = buf[pad:pad + n].view(x.shape)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    if entry == "ex":
        pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, util.layout_code(layout), ws)
    else:
        pkg.esc_convattn_forward(x, C_a, K, wl, wd, bd, out)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    assert bool((buf[:pad] == 7.0).all()) and bool((buf[pad + n:] == 7.0).all()), "write outside out"
    return x, out


def compare_full(pkg, oracle, d, C_a, K, dtype, layout, entry="ex", what="", unit_variance=False):
    import torch

    x, out = run_forward(pkg, d, C_a, K, dtype, layout, entry)
    ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
    got = util.to_host_nchw(out, layout)
    err = util.check_attention(got[:, :C_a], ref[:, :C_a], mag, dtype, what, unit_variance)
    # copy-through channels: bit-exact
    if C_a < d["x"].shape[1]:
        xs, os_ = (x, out) if layout == synth.NCHW else (x.permute(0, 3, 1, 2), out.permute(0, 3, 1, 2))
        assert torch.equal(xs[:, C_a:].contiguous().view(torch.int16 if dtype == synth.BF16 else torch.int32),
                           os_[:, C_a:].contiguous().view(torch.int16 if dtype == synth.BF16 else torch.int32))
    return err


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_dk_stage(pkg, oracle, dtype, layout):
    """GAP + linear layer on non-zero-mean data: dk within 1e-5 of max|dk| (fp32 arithmetic)."""
    import torch

    for (B, C, C_a, H, W) in [(3, 64, 16, 37, 53), (1, 64, 32, 120, 200), (2, 24, 8, 16, 16), (1, 20, 12, 9, 7),
                              (70, 32, 16, 8, 8),
                              (2, 192, 48, 33, 47), (1, 48, 24, 20, 30), (1, 144, 144, 12, 12)]:   # 6, 3 and 18 (or 12, 6, 36) chunks per pixel
        d = synth.make_inputs(B, C, C_a, H, W, 13, dtype, seed=B * 100 + H, channel_means=True)
        x = util.to_device(d["x"], dtype, layout)
        _, wd, bd = util.weights_to_device(d, dtype)
        dk = torch.full((B, C_a, 3, 3), float("nan"), device="cuda")
        ws = pkg.new_workspace(B, C_a, H, W, 13)
        for _ in range(2):  # twice: the arrival counters must be ready for reuse
            pkg.esc_convattn_dynkernel(x, C_a, wd, bd, dk, util.layout_code(layout), ws)
        torch.cuda.synchronize()
        ref = oracle.dynkernel(oracle.gap(d["x"], C_a), d["w_dyn"], d["b_dyn"])
        err = np.abs(dk.cpu().numpy().astype(np.float64) - ref).max()
        assert err <= 1e-5 * np.abs(ref).max(), (B, C, C_a, H, W, err)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_stencil_stage_explicit_dk(pkg, oracle, dtype, layout):
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 45, 70, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=77)
    dk = np.random.default_rng(5).uniform(-0.5, 0.5, size=(B, C_a, 3, 3)).astype(np.float32)
    x = util.to_device(d["x"], dtype, layout)
    wl, _, _ = util.weights_to_device(d, dtype)
    out = torch.empty_like(x)
    pkg.esc_convattn_stencil(x, C_a, K, wl, torch.from_numpy(dk).cuda(), out, util.layout_code(layout))
    torch.cuda.synchronize()
    ref, mag = oracle.stencil(d["x"], C_a, d["w_large"], dk, want_mag=True)
    got = util.to_host_nchw(out, layout)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, dtype, "stencil stage", unit_variance=True)
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])


EDGE_SHAPES = [
    # B, C, C_a, H, W, K
    (1, 64, 16, 5, 5, 13),      # H, W < K
    (2, 64, 16, 1, 40, 13),     # single row
    (2, 64, 16, 33, 1, 13),     # single column
    (1, 64, 16, 13, 13, 13),
    (3, 64, 16, 41, 83, 13),    # several tiles plus a ragged tail, odd W
    (1, 64, 16, 40, 40, 13),    # exactly one register tile
    (1, 64, 16, 80, 120, 13),   # whole tiles only
    (2, 16, 16, 30, 50, 13),    # C_a == C: nothing to copy through
    (2, 32, 8, 22, 36, 13),     # C_a = 8
    (1, 64, 32, 47, 61, 13),    # C_a = 32
    (1, 48, 16, 29, 31, 9),     # K = 9
    (1, 48, 16, 29, 31, 17),    # K = 17
    (1, 20, 12, 19, 23, 3),     # K = 3, odd channel counts
    (5, 64, 16, 64, 64, 13),    # small batch of training patches
    (1, 192, 48, 50, 70, 13),   # the paper's large model: C = 192, 48 attention channels (3 channel groups)
    (2, 48, 16, 45, 45, 13),    # ESC-FP width: C = 48
    (1, 272, 16, 41, 41, 13),   # 256 copy-through channels: narrowest copy box
    (1, 288, 16, 20, 20, 13),   # more copy-through channels than a TMA box holds: generic path
    (130, 32, 16, 40, 40, 13),  # many images of exactly one tile
    (1, 64, 16, 1200, 20, 13),  # tall and narrow
    (1, 64, 16, 17, 1500, 13),  # flat and wide
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", EDGE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_edge_shapes(pkg, oracle, shape, dtype, layout):
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, dtype, seed=sum(shape), per_image_scale=True, channel_means=True)
    compare_full(pkg, oracle, d, C_a, K, dtype, layout, what=str(shape))


TILE_SHAPES = [s for s in EDGE_SHAPES if s[5] == 13 and s[2] % 16 == 0 and s[1] - s[2] <= 256] + [
    (1, 64, 16, 16, 64, 13),    # exactly one 64x16 tile
    (2, 64, 16, 17, 65, 13),    # one pixel more in both directions
    (1, 64, 16, 293, 517, 13),  # ragged in both directions, over a hundred tiles of either geometry
    (3, 48, 32, 100, 129, 13),  # two channel groups, three images
]


@pytest.mark.parametrize("width", [40, 64])
@pytest.mark.parametrize("shape", TILE_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_both_tile_geometries(pkg, oracle, shape, width):
    """Every shape the TMA-staged kernel accepts, on each of its two tile geometries."""
    B, C, C_a, H, W, K = shape
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=sum(shape) + width, per_image_scale=True, channel_means=True)
    with tile_width(pkg, width):
        compare_full(pkg, oracle, d, C_a, K, synth.BF16, synth.NHWC, what=f"{shape} tile {width}")
        assert pkg.esc_convattn_last_path() == 2 and pkg.esc_convattn_last_tile_width() == width


def test_tile_choice_and_policy(pkg):
    """FP32 engine: the cost estimate takes 64x16 tiles for a batch of 64x64 patches and for maps with few tiles,
    40x40 tiles for the large maps; the override rejects widths that do not exist."""
    import torch

    def used(B, C, C_a, H, W):
        x = torch.zeros(B, H, W, C, dtype=torch.bfloat16, device="cuda")
        wl = torch.zeros(C_a, 13, 13, dtype=torch.bfloat16, device="cuda")
        dk = torch.zeros(B, C_a, 3, 3, device="cuda")
        ws = pkg.new_workspace(B, C_a, H, W, 13)
        pkg.esc_convattn_stencil(x, C_a, 13, wl, dk, torch.empty_like(x), pkg.ESC_NHWC, ws)
        torch.cuda.synchronize()
        assert pkg.esc_convattn_device_status(ws) == 0
        return pkg.esc_convattn_last_tile_width()

    pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
    try:
        assert used(64, 64, 16, 64, 64) == 64
        assert used(1, 64, 16, 90, 130) == 64
        assert used(1, 64, 16, 360, 640) == 40
        assert used(1, 64, 32, 1080, 1920) == 40
        with pytest.raises(pkg.EscError):
            pkg.esc_convattn_set_tile_width(48)
        assert used(1, 64, 16, 360, 640) == 40      # a rejected value leaves the policy alone
    finally:
        pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)


@pytest.mark.parametrize("wl_name", ["cfg1_64x64_f32", "cfg2_320x180_f32", "cfg3_640x360_bf16", "cfg4_b64_64x64_bf16"])
@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("means", [False, True], ids=["zero_mean", "channel_means"])
def test_forward_workloads_full(pkg, oracle, wl_name, layout, means):
    """The evaluation workloads, every output compared (the oracle needs a few seconds each)."""
    wl = synth.WORKLOADS_BY_NAME[wl_name]
    d = synth.make_workload(wl, channel_means=means)
    compare_full(pkg, oracle, d, wl.C_a, wl.K, wl.dtype, layout, what=wl_name,
                 unit_variance=not means and not wl.per_image_scale)


@pytest.mark.parametrize("wl_name,width", [("cfg3_640x360_bf16", 64), ("cfg4_b64_64x64_bf16", 40)])
def test_forward_workloads_other_geometry(pkg, oracle, wl_name, width):
    """The bf16 workloads on the tile geometry the cost estimate does not pick for them."""
    wl = synth.WORKLOADS_BY_NAME[wl_name]
    d = synth.make_workload(wl, channel_means=True)
    with tile_width(pkg, width):
        compare_full(pkg, oracle, d, wl.C_a, wl.K, wl.dtype, synth.NHWC, what=f"{wl_name} tile {width}")
        assert pkg.esc_convattn_last_tile_width() == width


def test_mandated_entry_fp32_nchw(pkg, oracle):
    wl = synth.WORKLOADS_BY_NAME["cfg1_64x64_f32"]
    d = synth.make_workload(wl, channel_means=True)
    compare_full(pkg, oracle, d, wl.C_a, wl.K, wl.dtype, synth.NCHW, entry="fixed", what="esc_convattn_forward")


@pytest.mark.parametrize("layout", LAYOUTS)
def test_forward_large_map_full(pkg, oracle, layout):
    """1920x1080, C_a = 32 bf16 in the launch configuration the benchmark times: every one of the 66 M
    attention outputs against the oracle, copy-through channels bit for bit.  On 148 SMs a CTA of the
    TMA-staged kernel walks 17 or 18 units here: the barrier phases wrap several times and the channel
    group (hence the weight table) changes inside a walk."""
    wl = synth.WORKLOADS_BY_NAME["cfg5_1920x1080_ca32_bf16"]
    d = synth.make_workload(wl, channel_means=True)
    compare_full(pkg, oracle, d, wl.C_a, wl.K, wl.dtype, layout, what="cfg5 full")


@pytest.mark.parametrize("width", [40, 64])
def test_forward_many_units_per_cta(pkg, oracle, width):
    """Eight images, two channel groups, 280x400: 1,120 units of 40x40 (1,792 of 64x16), i.e. seven to
    thirteen per CTA, with image and channel-group changes inside every CTA's walk; all outputs compared."""
    B, C, C_a, H, W, K = 8, 64, 32, 280, 400, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=2024 + width, per_image_scale=True, channel_means=True)
    with tile_width(pkg, width):
        compare_full(pkg, oracle, d, C_a, K, synth.BF16, synth.NHWC, what=f"many units, tile {width}")
        assert pkg.esc_convattn_last_path() == 2 and pkg.esc_convattn_last_tile_width() == width


@pytest.mark.parametrize("layout", LAYOUTS)
def test_bitwise_determinism_and_special_values(pkg, layout):
    """Run-to-run identical bits; NaN / -0 payloads in copy-through channels survive."""
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 90, 130, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=5, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, layout)
    xv = x.view(torch.int16)
    idt = (slice(None), slice(C_a, None)) if layout == synth.NCHW else (Ellipsis, slice(C_a, None))
    sub = xv[idt].contiguous().clone()
    sub.view(-1)[::97] = -32768          # -0.0
    sub.view(-1)[5::89] = 0x7FC1         # NaN with a payload
    xv[idt] = sub
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    outs = []
    for _ in range(3):
        out = torch.empty_like(x)
        pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, util.layout_code(layout), ws)
        torch.cuda.synchronize()
        outs.append(out.view(torch.int16).clone())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    assert torch.equal(outs[0][idt], xv[idt])


def test_host_entry_matches_device_entry(pkg):
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 60, 100, 13
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=15, channel_means=True)
    xh = torch.from_numpy(synth.to_layout(d["x"], synth.NHWC)).to(torch.bfloat16).pin_memory()
    wl, wd, bd = (torch.from_numpy(d[k]).to(torch.bfloat16) for k in ("w_large", "w_dyn", "b_dyn"))
    oh = torch.empty_like(xh).pin_memory()
    for _ in range(2):
        pkg.esc_convattn_forward_host(xh, C_a, K, wl, wd, bd, oh, pkg.ESC_NHWC)
    x = xh.cuda()
    out = torch.empty_like(x)
    ws = pkg.new_workspace(B, C_a, H, W, K)
    pkg.esc_convattn_forward_ex(x, C_a, K, wl.cuda(), wd.cuda(), bd.cuda(), out, pkg.ESC_NHWC, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.cpu().view(torch.int16), oh.view(torch.int16))


def test_host_submit_wait_two_slots_in_turn(pkg):
    """The asynchronous host-buffer pair: steps alternate between the two slots, every result equals the
    blocking call's bit for bit, and a second shape on the same slots works (buffers regrow)."""
    import torch

    with pytest.raises(pkg.EscError):
        pkg.esc_convattn_forward_host_wait(2)
    for (B, C, C_a, H, W, K) in [(1, 64, 16, 60, 100, 13), (2, 64, 16, 90, 130, 13)]:
        steps = []
        for seed in range(4):
            d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=300 + seed, channel_means=True)
            xh = torch.from_numpy(synth.to_layout(d["x"], synth.NHWC)).to(torch.bfloat16).pin_memory()
            w = [torch.from_numpy(d[k]).to(torch.bfloat16).pin_memory() for k in ("w_large", "w_dyn", "b_dyn")]
            ref = torch.empty_like(xh).pin_memory()
            pkg.esc_convattn_forward_host(xh, C_a, K, *w, ref, pkg.ESC_NHWC)
            steps.append((xh, w, ref, torch.zeros_like(xh).pin_memory()))
        for i, (xh, w, ref, out) in enumerate(steps):
            pkg.esc_convattn_forward_host_submit(i % 2, xh, C_a, K, *w, out, pkg.ESC_NHWC)
            if i > 0:
                pkg.esc_convattn_forward_host_wait((i - 1) % 2)
                assert torch.equal(steps[i - 1][3].view(torch.int16), steps[i - 1][2].view(torch.int16))
        pkg.esc_convattn_forward_host_wait((len(steps) - 1) % 2)
        assert torch.equal(steps[-1][3].view(torch.int16), steps[-1][2].view(torch.int16))


def test_two_streams_two_workspaces(pkg, oracle):
    """Calls on different streams with different workspaces may overlap on the GPU; each must still be right."""
    import torch

    B, C, C_a, H, W, K = 2, 64, 16, 120, 200, 13
    cases = []
    for seed in (1, 2):
        d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=9000 + seed, channel_means=True)
        x = util.to_device(d["x"], synth.BF16, synth.NHWC)
        wl, wd, bd = util.weights_to_device(d, synth.BF16)
        cases.append((d, x, wl, wd, bd, torch.empty_like(x), pkg.new_workspace(B, C_a, H, W, K), torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(5):
        for (d, x, wl, wd, bd, out, ws, st) in cases:
            pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, pkg.ESC_NHWC, ws, stream=st)
    torch.cuda.synchronize()
    for (d, x, wl, wd, bd, out, ws, st) in cases:
        assert pkg.esc_convattn_device_status(ws) == 0
        ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
        got = util.to_host_nchw(out, synth.NHWC)
        util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, "two streams")
        assert np.array_equal(got[:, C_a:], ref[:, C_a:])
