"""ctypes binding with the same names as include/esc_convattn.h (argument marshalling only).

Tensors are torch CUDA tensors (or, for the *_host call, CPU tensors); the binding passes their
data pointers, the logical sizes and the current stream.  Logical shape is always [B,C,H,W]:
an NCHW call takes a contiguous [B,C,H,W] tensor, an NHWC call a contiguous [B,H,W,C] tensor.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

ESC_F32, ESC_BF16 = 0, 1
ESC_NCHW, ESC_NHWC = 0, 1

_LIB_PATH = Path(__file__).resolve().parent / "lib" / "libesc_convattn.so"
_lib = None


class EscError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        text = esc_status_string(status)
        detail = esc_last_error() if self.status == 7 else ""
        super().__init__(f"{where}: status {self.status} ({text}){' -- ' + detail if detail else ''}")


def lib_path() -> Path:
    return _LIB_PATH


def lib():
    """The loaded C-ABI library; raises if it has not been built (no silent fall-back)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2503_06671_b200.build` "
                "(there is no CPU implementation to fall back to)")
        L = ctypes.CDLL(str(_LIB_PATH))
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.esc_convattn_forward.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp]
        L.esc_convattn_forward_ex.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_fused.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_workspace_bytes.argtypes = [i, i, i, i, i]
        L.esc_convattn_workspace_bytes.restype = sz
        L.esc_convattn_workspace_init.argtypes = [vp, sz, vp]
        L.esc_convattn_dynkernel.argtypes = [vp, i, i, i, i, i, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_mlp.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, i, vp, i, i, vp, sz, vp]
        L.esc_convattn_dynkernel_mlp.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp, i, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_pw.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_stencil_pw.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_dense.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_stencil_dense.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_variant.argtypes = [vp, i, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, vp, i, i, vp, sz, vp]
        L.esc_convattn_backward_workspace_bytes.argtypes = [i, i, i, i, i]
        L.esc_convattn_backward_workspace_bytes.restype = sz
        L.esc_convattn_backward.argtypes = [vp, vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_backward_mlp.argtypes = [vp, vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, i, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_backward_pw.argtypes = [vp, vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_backward_dense_workspace_bytes.argtypes = [i, i, i, i, i]
        L.esc_convattn_backward_dense_workspace_bytes.restype = sz
        L.esc_convattn_backward_dense.argtypes = [vp, vp, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_backward_variant.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, vp, vp, vp, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_conv_fuse_backward_workspace_bytes.argtypes = [i, i, i, i]
        L.esc_conv_fuse_backward_workspace_bytes.restype = sz
        L.esc_conv_fuse_backward.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_dynkernel_static.argtypes = [vp, i, i, i, i, i, vp, vp, vp, i, i, vp]
        L.esc_convattn_stencil.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, i, i, vp, sz, vp]
        L.esc_convattn_forward_host.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, i, i]
        L.esc_convattn_device_status.argtypes = [vp, vp]
        L.esc_convattn_selftest_bounded_wait.argtypes = [vp, vp]
        L.esc_convattn_forward_host_submit.argtypes = [i, vp, i, i, i, i, i, i, vp, vp, vp, vp, i, i]
        L.esc_convattn_forward_host_wait.argtypes = [i]
        L.esc_convattn_set_tile_width.argtypes = [i]
        L.esc_convattn_set_stencil_engine.argtypes = [i]
        L.esc_convattn_set_fused_stage1.argtypes = [i]
        L.esc_convattn_set_dense_engine.argtypes = [i]
        L.esc_status_string.argtypes = [i]
        L.esc_status_string.restype = ctypes.c_char_p
        L.esc_last_error.restype = ctypes.c_char_p
        for name in ("esc_convattn_forward", "esc_convattn_forward_ex", "esc_convattn_forward_fused", "esc_convattn_workspace_init",
                     "esc_convattn_dynkernel", "esc_convattn_dynkernel_static", "esc_convattn_forward_mlp", "esc_convattn_dynkernel_mlp", "esc_convattn_forward_pw", "esc_convattn_stencil_pw", "esc_convattn_forward_dense", "esc_convattn_stencil_dense", "esc_convattn_forward_variant", "esc_convattn_backward", "esc_convattn_backward_mlp", "esc_convattn_backward_pw", "esc_convattn_backward_dense", "esc_convattn_backward_variant", "esc_conv_fuse_backward", "esc_convattn_stencil", "esc_convattn_forward_host", "esc_convattn_forward_host_submit", "esc_convattn_forward_host_wait",
                     "esc_convattn_device_status", "esc_convattn_last_path", "esc_convattn_last_tile_width", "esc_convattn_set_tile_width", "esc_convattn_set_stencil_engine", "esc_convattn_set_fused_stage1", "esc_convattn_set_dense_engine", "esc_convattn_last_launches",
                     "esc_version"):
            getattr(L, name).restype = i
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch

    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(status, where):
    if status != 0:
        raise EscError(status, where)


def _dtype_code(t):
    import torch

    if t.dtype == torch.float32:
        return ESC_F32
    if t.dtype == torch.bfloat16:
        return ESC_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dims(x, layout):
    if x.dim() != 4 or not x.is_contiguous():
        raise ValueError("x must be a contiguous 4-D tensor in the memory order named by `layout`")
    if layout == ESC_NCHW:
        B, C, H, W = x.shape
    elif layout == ESC_NHWC:
        B, H, W, C = x.shape
    else:
        raise ValueError("layout")
    return int(B), int(C), int(H), int(W)


def esc_status_string(status) -> str:
    return lib().esc_status_string(int(status)).decode()


def esc_last_error() -> str:
    return lib().esc_last_error().decode()


def esc_version() -> int:
    return lib().esc_version()


def esc_convattn_last_path() -> int:
    return lib().esc_convattn_last_path()


def esc_convattn_last_tile_width() -> int:
    return lib().esc_convattn_last_tile_width()


def esc_convattn_set_tile_width(tile_width: int) -> None:
    _check(lib().esc_convattn_set_tile_width(int(tile_width)), "esc_convattn_set_tile_width")


ESC_ENGINE_AUTO, ESC_ENGINE_FP32, ESC_ENGINE_TENSOR = 0, 1, 2


def esc_convattn_set_dense_engine(engine: int) -> None:
    _check(lib().esc_convattn_set_dense_engine(int(engine)), "esc_convattn_set_dense_engine")


def esc_convattn_set_fused_stage1(on: bool) -> None:
    _check(lib().esc_convattn_set_fused_stage1(1 if on else 0), "esc_convattn_set_fused_stage1")


def esc_convattn_set_stencil_engine(engine: int) -> None:
    _check(lib().esc_convattn_set_stencil_engine(int(engine)), "esc_convattn_set_stencil_engine")


def esc_convattn_last_launches() -> int:
    return lib().esc_convattn_last_launches()


def esc_convattn_workspace_bytes(B, C_a, H, W, K) -> int:
    return int(lib().esc_convattn_workspace_bytes(B, C_a, H, W, K))


def esc_convattn_workspace_init(workspace, stream=None):
    _check(lib().esc_convattn_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                             _stream(stream)), "esc_convattn_workspace_init")


def new_workspace(B, C_a, H, W, K, device="cuda"):
    """Allocate (with torch) and initialise a workspace for the calls that take one."""
    import torch

    n = esc_convattn_workspace_bytes(B, C_a, H, W, K)
    if n == 0:
        raise ValueError("invalid problem size")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    esc_convattn_workspace_init(ws)
    return ws


def esc_convattn_forward(x, C_a, K, w_large, w_dyn, b_dyn, out, stream=None):
    """fp32 NCHW forward (library-owned scratch).  x, out: contiguous [B,C,H,W] float32 CUDA tensors."""
    B, C, H, W = _dims(x, ESC_NCHW)
    _check(lib().esc_convattn_forward(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn), _ptr(b_dyn),
                                      _ptr(out), _stream(stream)), "esc_convattn_forward")
    return out


def esc_convattn_forward_ex(x, C_a, K, w_large, w_dyn, b_dyn, out, layout, workspace, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_ex(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn), _ptr(b_dyn),
                                         _ptr(out), _dtype_code(x), layout, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_forward_ex")
    return out


def esc_convattn_forward_fused(x, C_a, K, w_large, w_dyn, b_dyn, w_fuse, b_fuse, residual, out, layout, workspace, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_fused(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn), _ptr(b_dyn), _ptr(w_fuse),
                                            _ptr(b_fuse), _ptr(residual), _ptr(out), _dtype_code(x), layout, _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_forward_fused")
    return out


def esc_convattn_dynkernel(x, C_a, w_dyn, b_dyn, dk_out, layout, workspace, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_dynkernel(_ptr(x), B, C, C_a, H, W, _ptr(w_dyn), _ptr(b_dyn), _ptr(dk_out),
                                        _dtype_code(x), layout, _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_dynkernel")
    return dk_out


def esc_convattn_forward_mlp(x, C_a, K, w_large, w_down, b_down, w_up, b_up, out, layout, workspace, stream=None):
    """Forward pass with the two-layer kernel estimator (hidden width = w_down.shape[0])."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_mlp(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_down), _ptr(b_down),
                                          _ptr(w_up), _ptr(b_up), int(w_down.shape[0]), _ptr(out), _dtype_code(x),
                                          layout, _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)),
           "esc_convattn_forward_mlp")
    return out


def esc_convattn_dynkernel_mlp(x, C_a, w_down, b_down, w_up, b_up, dk_out, layout, workspace, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_dynkernel_mlp(_ptr(x), B, C, C_a, H, W, _ptr(w_down), _ptr(b_down), _ptr(w_up),
                                            _ptr(b_up), int(w_down.shape[0]), _ptr(dk_out), _dtype_code(x), layout,
                                            _ptr(workspace), workspace.numel() * workspace.element_size(),
                                            _stream(stream)),
           "esc_convattn_dynkernel_mlp")
    return dk_out


def esc_convattn_forward_pw(x, C_a, K, w_large, w_point, w_dyn, b_dyn, out, layout, workspace, stream=None):
    """Forward pass in the decomposed form of Eq. 5: point-wise filter w_point [C_a,C_a], then the depth-wise stage."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_pw(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_point), _ptr(w_dyn),
                                         _ptr(b_dyn), _ptr(out), _dtype_code(x), layout, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_forward_pw")
    return out


def esc_convattn_stencil_pw(x, C_a, K, w_large, w_point, dk, out, layout, workspace=None, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_stencil_pw(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_point), _ptr(dk),
                                         _ptr(out), _dtype_code(x), layout, _ptr(workspace),
                                         0 if workspace is None else workspace.numel() * workspace.element_size(),
                                         _stream(stream)),
           "esc_convattn_stencil_pw")
    return out


def esc_convattn_forward_dense(x, C_a, K, w_dense, w_dyn, b_dyn, out, layout, workspace, stream=None):
    """Forward pass with the dense large kernel w_dense [C_a,C_a,K,K] (output channel, input channel, row, column)."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_dense(_ptr(x), B, C, C_a, H, W, K, _ptr(w_dense), _ptr(w_dyn), _ptr(b_dyn),
                                            _ptr(out), _dtype_code(x), layout, _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_forward_dense")
    return out


def esc_convattn_stencil_dense(x, C_a, K, w_dense, dk, out, layout, workspace=None, stream=None):
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_stencil_dense(_ptr(x), B, C, C_a, H, W, K, _ptr(w_dense), _ptr(dk), _ptr(out),
                                            _dtype_code(x), layout, _ptr(workspace),
                                            0 if workspace is None else workspace.numel() * workspace.element_size(),
                                            _stream(stream)),
           "esc_convattn_stencil_dense")
    return out


ESC_LK_DEPTHWISE, ESC_LK_DECOMPOSED, ESC_LK_DENSE = 0, 1, 2


def esc_convattn_backward_workspace_bytes(B, C_a, H, W, K) -> int:
    return int(lib().esc_convattn_backward_workspace_bytes(B, C_a, H, W, K))


def new_backward_workspace(B, C_a, H, W, K, device="cuda"):
    """Allocate (with torch) and zero a workspace for esc_convattn_backward."""
    import torch

    n = esc_convattn_backward_workspace_bytes(B, C_a, H, W, K)
    if n == 0:
        raise ValueError("invalid problem size, or K is not odd in 3 .. 13")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    esc_convattn_workspace_init(ws)
    return ws


def esc_convattn_backward(x, grad_out, C_a, K, w_large, w_dyn, b_dyn, grad_x, grad_w_large, grad_w_dyn, grad_b_dyn,
                          layout, workspace, stream=None):
    """Gradients of esc_convattn_forward_ex: grad_x like x; the three weight gradients are fp32 tensors or None."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_backward(_ptr(x), _ptr(grad_out), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn), _ptr(b_dyn),
                                       _ptr(grad_x), _ptr(grad_w_large), _ptr(grad_w_dyn), _ptr(grad_b_dyn),
                                       _dtype_code(x), layout, _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_backward")
    return grad_x


def esc_convattn_backward_mlp(x, grad_out, C_a, K, w_large, w_down, b_down, w_up, b_up, grad_x, grad_w_large, grad_w_down,
                              grad_b_down, grad_w_up, grad_b_up, layout, workspace, stream=None):
    """Gradients of esc_convattn_forward_mlp: grad_x like x; the five weight gradients are fp32 tensors or None."""
    B, C, H, W = _dims(x, layout)
    hidden = int(w_down.shape[0])
    _check(lib().esc_convattn_backward_mlp(_ptr(x), _ptr(grad_out), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_down), _ptr(b_down),
                                           _ptr(w_up), _ptr(b_up), hidden, _ptr(grad_x), _ptr(grad_w_large), _ptr(grad_w_down),
                                           _ptr(grad_b_down), _ptr(grad_w_up), _ptr(grad_b_up), _dtype_code(x), layout,
                                           _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_backward_mlp")
    return grad_x


def esc_convattn_backward_pw(x, grad_out, C_a, K, w_large, w_point, w_dyn, b_dyn, grad_x, grad_w_large, grad_w_point, grad_w_dyn,
                             grad_b_dyn, layout, workspace, stream=None):
    """Gradients of esc_convattn_forward_pw (decomposed form): grad_x like x; the four weight gradients are fp32 tensors or None."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_backward_pw(_ptr(x), _ptr(grad_out), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_point), _ptr(w_dyn),
                                          _ptr(b_dyn), _ptr(grad_x), _ptr(grad_w_large), _ptr(grad_w_point), _ptr(grad_w_dyn),
                                          _ptr(grad_b_dyn), _dtype_code(x), layout, _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_backward_pw")
    return grad_x


def esc_convattn_backward_dense_workspace_bytes(B, C_a, H, W, K) -> int:
    return int(lib().esc_convattn_backward_dense_workspace_bytes(B, C_a, H, W, K))


def new_backward_dense_workspace(B, C_a, H, W, K, device="cuda"):
    """Allocate (with torch) and zero a workspace for esc_convattn_backward_dense."""
    import torch

    n = esc_convattn_backward_dense_workspace_bytes(B, C_a, H, W, K)
    if n == 0:
        raise ValueError("invalid problem size, C_a is not 16, or K is not odd in 3 .. 13")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    esc_convattn_workspace_init(ws)
    return ws


def esc_convattn_backward_dense(x, grad_out, C_a, K, w_dense, w_dyn, b_dyn, grad_x, grad_w_dense, grad_w_dyn, grad_b_dyn, layout,
                                workspace, stream=None):
    """Gradients of esc_convattn_forward_dense: grad_x like x; the three weight gradients are fp32 tensors or None."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_backward_dense(_ptr(x), _ptr(grad_out), B, C, C_a, H, W, K, _ptr(w_dense), _ptr(w_dyn), _ptr(b_dyn),
                                             _ptr(grad_x), _ptr(grad_w_dense), _ptr(grad_w_dyn), _ptr(grad_b_dyn), _dtype_code(x),
                                             layout, _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_backward_dense")
    return grad_x


def esc_convattn_backward_variant(x, grad_out, C_a, K, large_kernel, w_large, w_point, w_down, b_down, w_up, b_up, grad_x,
                                  grad_w_large, grad_w_point, grad_w_down, grad_b_down, grad_w_up, grad_b_up, layout, workspace,
                                  stream=None):
    """Gradients of esc_convattn_forward_variant: any large-kernel form (ESC_LK_*) with either estimator (w_down None
    means one linear layer w_up, b_up).  Weight gradients are fp32 tensors or None."""
    B, C, H, W = _dims(x, layout)
    hidden = 0 if w_down is None else int(w_down.shape[0])
    _check(lib().esc_convattn_backward_variant(_ptr(x), _ptr(grad_out), B, C, C_a, H, W, K, int(large_kernel), _ptr(w_large),
                                               _ptr(w_point), _ptr(w_down), _ptr(b_down), _ptr(w_up), _ptr(b_up), hidden,
                                               _ptr(grad_x), _ptr(grad_w_large), _ptr(grad_w_point), _ptr(grad_w_down),
                                               _ptr(grad_b_down), _ptr(grad_w_up), _ptr(grad_b_up), _dtype_code(x), layout,
                                               _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_backward_variant")
    return grad_x


def esc_conv_fuse_backward_workspace_bytes(B, C, H, W) -> int:
    return int(lib().esc_conv_fuse_backward_workspace_bytes(B, C, H, W))


def esc_conv_fuse_backward(cat, grad_out, w_fuse, grad_cat, grad_w_fuse, grad_b_fuse, layout, workspace=None, stream=None):
    """Gradients of the closing 1x1 convolution: grad_cat like cat; grad_w_fuse [C,C] and grad_b_fuse [C] are fp32 tensors
    or None.  Without a workspace one is allocated with torch for the call."""
    import torch

    B, C, H, W = _dims(cat, layout)
    if workspace is None:
        n = esc_conv_fuse_backward_workspace_bytes(B, C, H, W)
        if n == 0:
            raise EscError(3, "esc_conv_fuse_backward_workspace_bytes")
        workspace = torch.empty(n, dtype=torch.uint8, device=cat.device)
    _check(lib().esc_conv_fuse_backward(_ptr(cat), _ptr(grad_out), B, C, H, W, _ptr(w_fuse), _ptr(grad_cat), _ptr(grad_w_fuse),
                                        _ptr(grad_b_fuse), _dtype_code(cat), layout, _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_conv_fuse_backward")
    return grad_cat


def esc_convattn_selftest_bounded_wait(workspace, stream=None):
    """Runs the library's bounded device-side wait on a barrier nothing signals (about a second): afterwards
    esc_convattn_device_status(workspace) returns 8 (ESC_DEV_TIMEOUT) once."""
    _check(lib().esc_convattn_selftest_bounded_wait(_ptr(workspace), _stream(stream)), "esc_convattn_selftest_bounded_wait")


def esc_convattn_forward_variant(x, C_a, K, large_kernel, w_large, w_point, w_down, b_down, w_up, b_up, out, layout,
                                 workspace, stream=None):
    """Any large-kernel form (ESC_LK_*) with either estimator: w_down None means one linear layer (w_up, b_up)."""
    B, C, H, W = _dims(x, layout)
    hidden = 0 if w_down is None else int(w_down.shape[0])
    _check(lib().esc_convattn_forward_variant(_ptr(x), B, C, C_a, H, W, K, int(large_kernel), _ptr(w_large), _ptr(w_point),
                                              _ptr(w_down), _ptr(b_down), _ptr(w_up), _ptr(b_up), hidden, _ptr(out),
                                              _dtype_code(x), layout, _ptr(workspace),
                                              workspace.numel() * workspace.element_size(), _stream(stream)),
           "esc_convattn_forward_variant")
    return out


def esc_convattn_dynkernel_static(x, C_a, w_dyn, b_dyn, dk_out, layout, stream=None):
    """Stage 1 without any device allocation: the scratch is a fixed array inside the library.

    For callers that may not call cudaMalloc (fixed-memory real-time loops, frameworks that own
    the allocator).  Limits and the sharing rule are in include/esc_convattn.h; sizes beyond the
    fixed scratch raise EscError with status 6."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_dynkernel_static(_ptr(x), B, C, C_a, H, W, _ptr(w_dyn), _ptr(b_dyn), _ptr(dk_out),
                                               _dtype_code(x), layout, _stream(stream)),
           "esc_convattn_dynkernel_static")
    return dk_out


def esc_convattn_stencil(x, C_a, K, w_large, dk, out, layout, workspace=None, stream=None):
    B, C, H, W = _dims(x, layout)
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().esc_convattn_stencil(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(dk), _ptr(out),
                                      _dtype_code(x), layout, _ptr(workspace), nbytes, _stream(stream)),
           "esc_convattn_stencil")
    return out


def esc_convattn_forward_host(x, C_a, K, w_large, w_dyn, b_dyn, out, layout):
    """Host-buffer call: CPU tensors in, CPU tensor out; copies and synchronisation happen inside."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_host(_ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn), _ptr(b_dyn),
                                           _ptr(out), _dtype_code(x), layout), "esc_convattn_forward_host")
    return out


def esc_convattn_forward_host_submit(slot, x, C_a, K, w_large, w_dyn, b_dyn, out, layout):
    """Asynchronous half of the host-buffer call: enqueue on slot 0 or 1 and return.  The CPU tensors must be
    pinned and stay untouched until esc_convattn_forward_host_wait(slot) returns."""
    B, C, H, W = _dims(x, layout)
    _check(lib().esc_convattn_forward_host_submit(int(slot), _ptr(x), B, C, C_a, H, W, K, _ptr(w_large), _ptr(w_dyn),
                                                  _ptr(b_dyn), _ptr(out), _dtype_code(x), layout),
           "esc_convattn_forward_host_submit")


def esc_convattn_forward_host_wait(slot) -> None:
    _check(lib().esc_convattn_forward_host_wait(int(slot)), "esc_convattn_forward_host_wait")


def esc_convattn_device_status(workspace, stream=None) -> int:
    return lib().esc_convattn_device_status(_ptr(workspace), _stream(stream))
