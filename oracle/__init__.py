"""TEST INFRASTRUCTURE: CPU oracle for the ConvAttn forward pass (see convattn_ref.c).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may use
this package.  It imports nothing from the CUDA package.
"""
from .convattn_oracle import (  # noqa: F401
    build,
    forward,
    gap,
    dynkernel,
    dynkernel_mlp,
    forward_mlp,
    stencil,
    backward,
    backward_mlp,
    backward_pw,
    backward_dense,
    backward_dense_points,
    backward_variant,
    stencil_dense,
    forward_dense,
    pointwise,
    stencil_pw,
    forward_pw,
    points,
    fuse,
    forward_fused,
    fuse_backward,
    set_threads,
    max_threads,
)
