"""TEST INFRASTRUCTURE: ctypes loader for the plain-C ConvAttn oracle.

The arithmetic lives in ``convattn_ref.c`` (direct nested loops, fp64
accumulation, ESC paper Section 3.3, Eq. 4 / Eq. 5).  This module only compiles
that file with gcc, marshals numpy arrays in and out, and sets the OpenMP thread
count used by the timing harness.  Logical layout everywhere is dense
``[B, C, H, W]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "convattn_ref.c"
_LIB = _HERE / "libconvattn_ref.so"
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i64p = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> Path:
    """Compile convattn_ref.c into a shared object next to it (gcc -O2 -fopenmp)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(".so.tmp%d" % os.getpid())
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _omp = None
        for name in ("libgomp.so.1",):
            try:
                _omp = ctypes.CDLL(name)
                break
            except OSError:
                pass
        _lib._omp = _omp
    return _lib


def max_threads() -> int:
    """Cores this process may run on (what OpenMP would use by default)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def set_threads(n: int) -> None:
    lib = _load()
    if lib._omp is not None:
        lib._omp.omp_set_num_threads(int(n))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_f64p)


def _dims(x, C_a, K):
    B, C, H, W = (int(v) for v in x.shape)
    assert 0 < C_a <= C and K % 2 == 1 and K >= 1
    return B, C, H, W


def gap(x, C_a):
    """g[B,C_a]: per-image, per-channel mean of the first C_a channels."""
    x, xp = _f32(x)
    B, C, H, W = (int(v) for v in x.shape)
    g = np.empty((B, C_a), dtype=np.float64)
    _load().convattn_ref_gap(xp, B, C, C_a, H, W, g.ctypes.data_as(_f64p))
    return g


def dynkernel(g, w_dyn, b_dyn):
    """dk[B,C_a,3,3] = W_dyn g + b_dyn, output index o = c*9 + i*3 + j."""
    g, gp = _f64(g)
    B, C_a = (int(v) for v in g.shape)
    w_dyn, wp = _f64(w_dyn)
    b_dyn, bp = _f64(b_dyn)
    assert w_dyn.shape == (9 * C_a, C_a) and b_dyn.shape == (9 * C_a,)
    dk = np.empty((B, C_a, 3, 3), dtype=np.float64)
    _load().convattn_ref_dynkernel(gp, B, C_a, wp, bp, dk.ctypes.data_as(_f64p))
    return dk


def dynkernel_mlp(g, w_down, b_down, w_up, b_up, want_hidden=False):
    """dk[B,C_a,3,3] = W_up GELU(W_down g + b_down) + b_up (Eq. 4 line 2 as written, exact-erf GELU)."""
    g, gp = _f64(g)
    B, C_a = (int(v) for v in g.shape)
    w_down, wdp = _f64(w_down)
    b_down, bdp = _f64(b_down)
    w_up, wup = _f64(w_up)
    b_up, bup = _f64(b_up)
    h = int(w_down.shape[0])
    assert 1 <= h <= 256
    assert w_down.shape == (h, C_a) and b_down.shape == (h,)
    assert w_up.shape == (9 * C_a, h) and b_up.shape == (9 * C_a,)
    dk = np.empty((B, C_a, 3, 3), dtype=np.float64)
    hid = np.empty((B, h), dtype=np.float64)
    _load().convattn_ref_dynkernel_mlp(gp, B, C_a, h, wdp, bdp, wup, bup, hid.ctypes.data_as(_f64p),
                                       dk.ctypes.data_as(_f64p))
    return (dk, hid) if want_hidden else dk


def forward_mlp(x, C_a, w_large, w_down, b_down, w_up, b_up, want_mag=False, want_dk=False):
    """Whole forward with the two-layer estimator: GAP, dynkernel_mlp, stencil, in that order."""
    dk = dynkernel_mlp(gap(x, C_a), w_down, b_down, w_up, b_up)
    res = stencil(x, C_a, w_large, dk, want_mag=want_mag)
    res = list(res) if want_mag else [res]
    if want_dk:
        res.append(dk)
    return res[0] if len(res) == 1 else tuple(res)


def pointwise(x, C_a, w_point, want_abs=False):
    """xm[B,C_a,H,W] = 1x1 convolution of the attention channels with w_point[C_a,C_a] (Eq. 5, LK^c), no bias."""
    x, xp = _f32(x)
    B, C, H, W = (int(v) for v in x.shape)
    w_point, wp = _f64(w_point)
    assert w_point.shape == (C_a, C_a) and C_a <= C
    xm = np.empty((B, C_a, H, W), dtype=np.float64)
    xabs = np.empty((B, C_a, H, W), dtype=np.float64) if want_abs else None
    _load().convattn_ref_pointwise(xp, B, C, C_a, H, W, wp, xm.ctypes.data_as(_f64p),
                                   xabs.ctypes.data_as(_f64p) if want_abs else None)
    return (xm, xabs) if want_abs else xm


def stencil_pw(x, C_a, w_large, w_point, dk, want_mag=False):
    """Decomposed form of Eq. 5 with an explicit dk: (F_att * LK^c) * (ZP(dk) + LK^s); other channels copied."""
    x, xp = _f32(x)
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    assert w_large.shape == (C_a, K, K)
    dk, dp = _f64(dk)
    assert dk.size == B * C_a * 9
    xm, xabs = pointwise(x, C_a, w_point, want_abs=True)
    out = np.empty((B, C, H, W), dtype=np.float64)
    mag = np.empty((B, C_a, H, W), dtype=np.float64) if want_mag else None
    _load().convattn_ref_stencil_mixed(
        xp, xm.ctypes.data_as(_f64p), xabs.ctypes.data_as(_f64p), B, C, C_a, H, W, K, wp, dp,
        out.ctypes.data_as(_f64p), mag.ctypes.data_as(_f64p) if want_mag else None,
    )
    return (out, mag) if want_mag else out


def forward_pw(x, C_a, w_large, w_point, w_dyn, b_dyn, want_mag=False, want_dk=False):
    """Whole forward in the decomposed form: dk from GAP(F_att) (one-layer estimator), then stencil_pw."""
    dk = dynkernel(gap(x, C_a), w_dyn, b_dyn)
    res = stencil_pw(x, C_a, w_large, w_point, dk, want_mag=want_mag)
    res = list(res) if want_mag else [res]
    if want_dk:
        res.append(dk)
    return res[0] if len(res) == 1 else tuple(res)


def stencil_dense(x, C_a, w_dense, dk, want_mag=False):
    """Dense large kernel w_dense[C_a,C_a,K,K] (out, in, row, col) plus the depth-wise dynamic 3x3 kernel dk."""
    x, xp = _f32(x)
    w_dense, wp = _f64(w_dense)
    K = int(w_dense.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    assert w_dense.shape == (C_a, C_a, K, K)
    dk, dp = _f64(dk)
    assert dk.size == B * C_a * 9
    out = np.empty((B, C, H, W), dtype=np.float64)
    mag = np.empty((B, C_a, H, W), dtype=np.float64) if want_mag else None
    _load().convattn_ref_stencil_dense(xp, B, C, C_a, H, W, K, wp, dp, out.ctypes.data_as(_f64p),
                                       mag.ctypes.data_as(_f64p) if want_mag else None)
    return (out, mag) if want_mag else out


def forward_dense(x, C_a, w_dense, w_dyn, b_dyn, want_mag=False, want_dk=False):
    """Whole forward with the dense large kernel: dk from GAP(F_att) (one-layer estimator), then stencil_dense."""
    dk = dynkernel(gap(x, C_a), w_dyn, b_dyn)
    res = stencil_dense(x, C_a, w_dense, dk, want_mag=want_mag)
    res = list(res) if want_mag else [res]
    if want_dk:
        res.append(dk)
    return res[0] if len(res) == 1 else tuple(res)


def backward(x, grad_out, C_a, w_large, w_dyn, b_dyn):
    """Gradients of forward(x, ...) contracted with grad_out: returns (gx [B,C,H,W], g_w_large [C_a,K,K],
    g_w_dyn [9*C_a,C_a], g_b_dyn [9*C_a])."""
    x, xp = _f32(x)
    go, gp = _f32(grad_out)
    assert go.shape == x.shape
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    w_dyn, wdp = _f64(w_dyn)
    b_dyn, bdp = _f64(b_dyn)
    gx = np.empty((B, C, H, W), dtype=np.float64)
    glk = np.empty((C_a, K, K), dtype=np.float64)
    gw = np.empty((9 * C_a, C_a), dtype=np.float64)
    gb = np.empty((9 * C_a,), dtype=np.float64)
    _load().convattn_ref_backward(xp, gp, B, C, C_a, H, W, K, wp, wdp, bdp, gx.ctypes.data_as(_f64p),
                                  glk.ctypes.data_as(_f64p), gw.ctypes.data_as(_f64p), gb.ctypes.data_as(_f64p))
    return gx, glk, gw, gb


def backward_mlp(x, grad_out, C_a, w_large, w_down, b_down, w_up, b_up):
    """Gradients of forward_mlp(x, ...) contracted with grad_out: returns (gx [B,C,H,W], g_w_large [C_a,K,K],
    g_w_down [h,C_a], g_b_down [h], g_w_up [9*C_a,h], g_b_up [9*C_a])."""
    x, xp = _f32(x)
    go, gp = _f32(grad_out)
    assert go.shape == x.shape
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    assert K >= 3
    B, C, H, W = _dims(x, C_a, K)
    w_down, wdp = _f64(w_down)
    b_down, bdp = _f64(b_down)
    w_up, wup = _f64(w_up)
    b_up, bup = _f64(b_up)
    h = int(w_down.shape[0])
    assert w_down.shape == (h, C_a) and b_down.shape == (h,) and w_up.shape == (9 * C_a, h) and b_up.shape == (9 * C_a,)
    gx = np.empty((B, C, H, W), dtype=np.float64)
    glk = np.empty((C_a, K, K), dtype=np.float64)
    gwd = np.empty((h, C_a), dtype=np.float64)
    gbd = np.empty((h,), dtype=np.float64)
    gwu = np.empty((9 * C_a, h), dtype=np.float64)
    gbu = np.empty((9 * C_a,), dtype=np.float64)
    _load().convattn_ref_backward_mlp(xp, gp, B, C, C_a, H, W, K, wp, h, wdp, bdp, wup, bup, *(a.ctypes.data_as(_f64p)
                                      for a in (gx, glk, gwd, gbd, gwu, gbu)))
    return gx, glk, gwd, gbd, gwu, gbu


def backward_pw(x, grad_out, C_a, w_large, w_point, w_dyn, b_dyn):
    """Gradients of forward_pw(x, ...) contracted with grad_out: returns (gx [B,C,H,W], g_w_large [C_a,K,K],
    g_w_point [C_a,C_a], g_w_dyn [9*C_a,C_a], g_b_dyn [9*C_a])."""
    x, xp = _f32(x)
    go, gp = _f32(grad_out)
    assert go.shape == x.shape
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    assert K >= 3
    B, C, H, W = _dims(x, C_a, K)
    w_point, wpp = _f64(w_point)
    assert w_point.shape == (C_a, C_a)
    w_dyn, wdp = _f64(w_dyn)
    b_dyn, bdp = _f64(b_dyn)
    gx = np.empty((B, C, H, W), dtype=np.float64)
    glk = np.empty((C_a, K, K), dtype=np.float64)
    gwp = np.empty((C_a, C_a), dtype=np.float64)
    gw = np.empty((9 * C_a, C_a), dtype=np.float64)
    gb = np.empty((9 * C_a,), dtype=np.float64)
    _load().convattn_ref_backward_pw(xp, gp, B, C, C_a, H, W, K, wp, wpp, wdp, bdp, *(a.ctypes.data_as(_f64p)
                                     for a in (gx, glk, gwp, gw, gb)))
    return gx, glk, gwp, gw, gb


def backward_dense(x, grad_out, C_a, w_dense, w_dyn, b_dyn):
    """Gradients of forward_dense(x, ...) contracted with grad_out: returns (gx [B,C,H,W], g_w_dense [C_a,C_a,K,K],
    g_w_dyn [9*C_a,C_a], g_b_dyn [9*C_a])."""
    x, xp = _f32(x)
    go, gp = _f32(grad_out)
    assert go.shape == x.shape
    w_dense, wp = _f64(w_dense)
    K = int(w_dense.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    assert w_dense.shape == (C_a, C_a, K, K)
    w_dyn, wdp = _f64(w_dyn)
    b_dyn, bdp = _f64(b_dyn)
    gx = np.empty((B, C, H, W), dtype=np.float64)
    gwd = np.empty((C_a, C_a, K, K), dtype=np.float64)
    gw = np.empty((9 * C_a, C_a), dtype=np.float64)
    gb = np.empty((9 * C_a,), dtype=np.float64)
    _load().convattn_ref_backward_dense(xp, gp, B, C, C_a, H, W, K, wp, wdp, bdp, *(a.ctypes.data_as(_f64p)
                                        for a in (gx, gwd, gw, gb)))
    return gx, gwd, gw, gb


def backward_dense_points(x, grad_out, C_a, K, idx):
    """Selected entries of the dense kernel's gradient (flat indices into [C_a,C_a,K,K]): returns (values, magnitudes)."""
    x, xp = _f32(x)
    go, gp = _f32(grad_out)
    assert go.shape == x.shape
    B, C, H, W = _dims(x, C_a, K)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    assert idx.ndim == 1 and (idx >= 0).all() and (idx < C_a * C_a * K * K).all()
    vals = np.empty(idx.shape, dtype=np.float64)
    mags = np.empty(idx.shape, dtype=np.float64)
    _load().convattn_ref_backward_dense_points(xp, gp, B, C, C_a, H, W, K, ctypes.c_int64(idx.size),
                                               idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                                               vals.ctypes.data_as(_f64p), mags.ctypes.data_as(_f64p))
    return vals, mags


def backward_variant(x, grad_out, C_a, large_kernel, w_large, w_point, w_down, b_down, w_up, b_up):
    """Gradients of a forward with any large-kernel form ("depthwise", "pw", "dense") and the two-layer estimator of
    Eq. 4 line 2, by the chain rule in two steps.  (1) Per image, with the generator frozen at that image's dk
    (W_dyn = 0, b_dyn = dk[b]) the one-layer backward of the form gives the stencil stage's part of gx, the large
    kernel's gradients (summed over images) and, as its g_b_dyn, dL/ddk[b].  (2) Through the estimator,
    t = W_down g + b_down, a = phi(t), dk = W_up a + b_up:
        g_bu = sum_b g_dk      g_Wu = sum_b g_dk a^T      g_a = W_up^T g_dk      g_t = g_a * phi'(t)
        g_bd = sum_b g_t       g_Wd = sum_b g_t g^T       g_g = W_down^T g_t     gx[b, :C_a] += g_g[b] / (H W)
    with phi'(t) = Phi(t) + t n(t).  Returns (gx, g_w_large, g_w_point or None, g_w_down, g_b_down, g_w_up, g_b_up)."""
    import math

    xa = np.ascontiguousarray(x, dtype=np.float32)
    go = np.ascontiguousarray(grad_out, dtype=np.float32)
    B, C, H, W = xa.shape
    w_down = np.asarray(w_down, dtype=np.float64); b_down = np.asarray(b_down, dtype=np.float64)
    w_up = np.asarray(w_up, dtype=np.float64); b_up = np.asarray(b_up, dtype=np.float64)
    g = gap(xa, C_a)
    dk = dynkernel_mlp(g, w_down, b_down, w_up, b_up).reshape(B, 9 * C_a)
    zero_w = np.zeros((9 * C_a, C_a))
    gx = np.empty((B, C, H, W), dtype=np.float64)
    g_large = None
    g_point = None
    g_dk = np.empty((B, 9 * C_a))
    for b in range(B):
        xb, gb_ = xa[b:b + 1], go[b:b + 1]
        if large_kernel == "depthwise":
            r = backward(xb, gb_, C_a, w_large, zero_w, dk[b])
            gxb, glb, gdkb = r[0], r[1], r[3]
        elif large_kernel == "pw":
            r = backward_pw(xb, gb_, C_a, w_large, w_point, zero_w, dk[b])
            gxb, glb, gdkb = r[0], r[1], r[4]
            g_point = r[2] if g_point is None else g_point + r[2]
        elif large_kernel == "dense":
            r = backward_dense(xb, gb_, C_a, w_large, zero_w, dk[b])
            gxb, glb, gdkb = r[0], r[1], r[3]
        else:
            raise ValueError(large_kernel)
        gx[b] = gxb[0]
        g_large = glb if g_large is None else g_large + glb
        g_dk[b] = gdkb
    t = g @ w_down.T + b_down                                           # [B, h]
    Phi = np.vectorize(lambda v: 0.5 * math.erfc(-v / math.sqrt(2.0)))(t)
    a = t * Phi
    dphi = Phi + t * np.exp(-0.5 * t * t) / math.sqrt(2.0 * math.pi)
    g_bu = g_dk.sum(axis=0)
    g_wu = g_dk.T @ a
    g_t = (g_dk @ w_up) * dphi
    g_bd = g_t.sum(axis=0)
    g_wd = g_t.T @ g
    g_g = g_t @ w_down                                                  # [B, C_a]
    gx[:, :C_a] += (g_g / (float(H) * float(W)))[:, :, None, None]
    return gx, g_large, g_point, g_wd, g_bd, g_wu, g_bu


def stencil(x, C_a, w_large, dk, rows=None, want_mag=False):
    """Stencil stage with an explicit dk[B,C_a,3,3]; rows=(y0,y1) restricts the output rows."""
    x, xp = _f32(x)
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    assert w_large.shape == (C_a, K, K)
    dk, dp = _f64(dk)
    assert dk.size == B * C_a * 9
    y0, y1 = (0, H) if rows is None else (int(rows[0]), int(rows[1]))
    assert 0 <= y0 <= y1 <= H
    out = np.empty((B, C, y1 - y0, W), dtype=np.float64)
    mag = np.empty((B, C_a, y1 - y0, W), dtype=np.float64) if want_mag else None
    _load().convattn_ref_stencil(
        xp, B, C, C_a, H, W, K, wp, dp, y0, y1, out.ctypes.data_as(_f64p),
        mag.ctypes.data_as(_f64p) if want_mag else None,
    )
    return (out, mag) if want_mag else out


def forward(x, C_a, w_large, w_dyn, b_dyn, want_mag=False, want_dk=False):
    """Whole ConvAttn forward.  Returns out[B,C,H,W] (fp64) and, on request, mag and dk."""
    x, xp = _f32(x)
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    assert w_large.shape == (C_a, K, K)
    w_dyn, wdp = _f64(w_dyn)
    b_dyn, bdp = _f64(b_dyn)
    assert w_dyn.shape == (9 * C_a, C_a) and b_dyn.shape == (9 * C_a,)
    out = np.empty((B, C, H, W), dtype=np.float64)
    g = np.empty((B, C_a), dtype=np.float64)
    dk = np.empty((B, C_a, 3, 3), dtype=np.float64)
    mag = np.empty((B, C_a, H, W), dtype=np.float64) if want_mag else None
    _load().convattn_ref_forward(
        xp, B, C, C_a, H, W, K, wp, wdp, bdp, out.ctypes.data_as(_f64p), g.ctypes.data_as(_f64p),
        dk.ctypes.data_as(_f64p), mag.ctypes.data_as(_f64p) if want_mag else None,
    )
    res = [out]
    if want_mag:
        res.append(mag)
    if want_dk:
        res.append(dk)
    return res[0] if len(res) == 1 else tuple(res)


def points(x, C_a, w_large, w_dyn, b_dyn, flat_idx, want_mag=False):
    """Outputs at the given flat indices of out[B,C,H,W], computed one by one."""
    x, xp = _f32(x)
    w_large, wp = _f64(w_large)
    K = int(w_large.shape[-1])
    B, C, H, W = _dims(x, C_a, K)
    dk = dynkernel(gap(x, C_a), w_dyn, b_dyn)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    assert idx.ndim == 1 and (idx >= 0).all() and (idx < x.size).all()
    vals = np.empty(idx.shape, dtype=np.float64)
    mags = np.empty(idx.shape, dtype=np.float64)
    _load().convattn_ref_points(
        xp, B, C, C_a, H, W, K, wp, dk.ctypes.data_as(_f64p), ctypes.c_int64(idx.size),
        idx.ctypes.data_as(_i64p), vals.ctypes.data_as(_f64p), mags.ctypes.data_as(_f64p),
    )
    return (vals, mags) if want_mag else vals


def fuse(cat, w_fuse, b_fuse=None, residual=None, want_mag=False):
    """Conv_fuse (1x1 over all C channels, Eq. 4 line 4) of a concatenated map cat[B,C,H,W] (fp64), plus bias and the
    block's residual (Eq. 3 line 3) when given."""
    cat = np.ascontiguousarray(cat, dtype=np.float64)
    B, C, H, W = cat.shape
    w_fuse, wp = _f64(w_fuse)
    assert w_fuse.shape == (C, C)
    bp = None
    if b_fuse is not None:
        b_fuse, bp = _f64(b_fuse)
        assert b_fuse.shape == (C,)
    rp = None
    if residual is not None:
        residual, rp = _f32(residual)
        assert residual.shape == cat.shape
    out = np.empty_like(cat)
    mag = np.empty_like(cat) if want_mag else None
    _load().convattn_ref_fuse(cat.ctypes.data_as(_f64p), B, C, H, W, wp, bp, rp, out.ctypes.data_as(_f64p),
                              mag.ctypes.data_as(_f64p) if want_mag else None)
    return (out, mag) if want_mag else out


def fuse_backward(cat, grad_out, w_fuse, want_mag=False):
    """Gradients of fuse(cat, w_fuse, b_fuse, residual) contracted with grad_out: returns (g_cat [B,C,H,W],
    g_w_fuse [C,C], g_b_fuse [C]); the residual's gradient is grad_out itself."""
    cat, cp = _f32(cat)
    go, gp = _f32(grad_out)
    assert go.shape == cat.shape
    B, C, H, W = (int(v) for v in cat.shape)
    w_fuse, wp = _f64(w_fuse)
    assert w_fuse.shape == (C, C)
    g_cat = np.empty((B, C, H, W), dtype=np.float64)
    g_w = np.empty((C, C), dtype=np.float64)
    g_b = np.empty((C,), dtype=np.float64)
    mag = np.empty((B, C, H, W), dtype=np.float64) if want_mag else None
    _load().convattn_ref_fuse_backward(cp, gp, B, C, H, W, wp, g_cat.ctypes.data_as(_f64p), g_w.ctypes.data_as(_f64p),
                                       g_b.ctypes.data_as(_f64p), mag.ctypes.data_as(_f64p) if want_mag else None)
    return (g_cat, g_w, g_b, mag) if want_mag else (g_cat, g_w, g_b)


def forward_fused(x, C_a, w_large, w_dyn, b_dyn, w_fuse, b_fuse=None, residual=None, want_mag=False, want_cat=False):
    """The whole module of Eq. 4 including its last line: ConvAttn stages, then Conv_fuse (+ residual)."""
    cat = forward(x, C_a, w_large, w_dyn, b_dyn)
    res = fuse(cat, w_fuse, b_fuse, residual, want_mag=want_mag)
    if want_cat:
        return (*res, cat) if want_mag else (res, cat)
    return res
