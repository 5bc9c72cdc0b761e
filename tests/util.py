"""Helpers shared by the GPU parity tests: tensor marshalling and the error bars."""
import numpy as np

from paper_2503_06671_b200 import synth

# Tolerances (stated where they are used, too):
#  fp32 storage : max|err| <= 1e-5 * max|ref|   and   |err| <= 1e-5 * sum|w*x| per output
#                 (the forward-error form: 178 fp32 FMAs have a rounding error of at most
#                  ~178 * 2^-24 = 1.1e-5 of sum|w*x| in the worst case, ~1e-6 in practice)
#  bf16 storage : |err| <= 2e-2 absolute on unit-variance data and |err| <= 1e-2 * max(|ref|, 1)
#                 (one round-to-nearest bf16 rounding of the fp32 sum: 2^-9 relative = 3.9e-3)
F32_REL = 1e-5
BF16_ABS = 2e-2
BF16_REL = 1e-2


def torch_dtype(dtype):
    import torch

    return torch.bfloat16 if dtype == synth.BF16 else torch.float32


def to_device(a_nchw, dtype, layout):
    """float32 logical [B,C,H,W] numpy (already rounded to dtype) -> CUDA tensor in memory order `layout`."""
    import torch

    return torch.from_numpy(synth.to_layout(a_nchw, layout)).to("cuda", torch_dtype(dtype))


def weights_to_device(d, dtype):
    import torch

    return tuple(torch.from_numpy(d[k]).to("cuda", torch_dtype(dtype)) for k in ("w_large", "w_dyn", "b_dyn"))


def to_host_nchw(t, layout):
    return synth.from_layout(t.float().cpu().numpy(), layout)


def layout_code(layout):
    from paper_2503_06671_b200 import ESC_NCHW, ESC_NHWC

    return ESC_NHWC if layout == synth.NHWC else ESC_NCHW


def check_attention(got, ref, mag, dtype, what="", unit_variance=False):
    """got/ref/mag: arrays of attention-channel outputs (any matching shape).

    The absolute bf16 bar is stated for unit-variance data; inputs with added channel means or
    per-image scales have larger outputs, so there only the relative and per-element bars apply."""
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    if dtype == synth.F32:
        scale = np.abs(ref).max()
        assert err.max() <= F32_REL * scale, f"{what}: max|err|={err.max():.3e} vs {F32_REL}*max|ref|={scale:.3e}"
        fe = (err / np.maximum(mag, 1e-30)).max()
        assert fe <= F32_REL, f"{what}: forward error {fe:.3e} > {F32_REL}"
    else:
        if unit_variance:
            assert err.max() <= BF16_ABS, f"{what}: max|err|={err.max():.3e} > {BF16_ABS}"
        rel = (err / np.maximum(np.abs(ref), 1.0)).max()
        assert rel <= BF16_REL, f"{what}: rel err {rel:.3e} > {BF16_REL}"
        # tighter, scale-aware bar: half a bf16 ulp of the result plus fp32 accumulation noise
        bar = 2.0 ** -8 * np.abs(ref) + 1e-5 * mag + 1e-30
        assert (err <= bar).all(), f"{what}: {int((err > bar).sum())} outputs beyond one bf16 rounding"
    return float(err.max())
