"""B200 (sm_100a) ConvAttn forward: thin Python binding over the C-ABI CUDA library.

Every step of the operation (ESC paper, Section 3.3, Eq. 4) runs in the library's kernels;
this package only marshals arguments.  PyTorch is used for device memory and streams.
There is no CPU fall-back: calls raise if the CUDA library is missing or no GPU is present.
"""
from . import synth  # noqa: F401  (seeded inputs; no ConvAttn arithmetic)
from .binding import (  # noqa: F401
    EscError,
    ESC_F32, ESC_BF16, ESC_NCHW, ESC_NHWC,
    lib, lib_path,
    esc_convattn_forward,
    esc_convattn_forward_ex,
    esc_convattn_forward_host,
    esc_convattn_dynkernel,
    esc_convattn_dynkernel_static,
    esc_convattn_stencil,
    esc_convattn_workspace_bytes,
    esc_convattn_workspace_init,
    esc_convattn_device_status,
    esc_convattn_forward_host_submit,
    esc_convattn_forward_host_wait,
    esc_convattn_forward_dense,
    esc_convattn_stencil_dense,
    esc_convattn_forward_variant,
    ESC_LK_DEPTHWISE, ESC_LK_DECOMPOSED, ESC_LK_DENSE,
    esc_convattn_backward,
    esc_convattn_backward_mlp,
    esc_convattn_backward_pw,
    esc_convattn_backward_workspace_bytes,
    new_backward_workspace,
    esc_convattn_forward_mlp,
    esc_convattn_forward_fused,
    esc_convattn_forward_pw,
    esc_convattn_stencil_pw,
    esc_convattn_dynkernel_mlp,
    esc_convattn_last_path,
    esc_convattn_last_tile_width,
    esc_convattn_set_tile_width,
    esc_convattn_set_stencil_engine,
    esc_convattn_set_fused_stage1,
    esc_convattn_set_dense_engine,
    ESC_ENGINE_AUTO, ESC_ENGINE_FP32, ESC_ENGINE_TENSOR,
    esc_convattn_last_launches,
    esc_status_string,
    esc_last_error,
    esc_version,
    new_workspace,
)
