"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2503_06671_b200 import build, lib

    build.build()
    return lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "esc_convattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(esc_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared_symbols()
    assert "esc_convattn_forward" in names and "esc_convattn_forward_ex" in names and len(names) >= 12
    for n in names:
        assert hasattr(L, n), n


def test_binding_has_the_same_names(L):
    import paper_2503_06671_b200 as pkg

    for n in _declared_symbols():
        assert hasattr(pkg, n), n


def test_version_and_strings(L):
    assert L.esc_version() >= 100
    assert L.esc_status_string(0) == b"ok"
    assert b"overlaps" in L.esc_status_string(5)
    assert L.esc_status_string(12345) == b"unknown status"


def test_workspace_bytes(L):
    n = L.esc_convattn_workspace_bytes(1, 16, 360, 640, 13)
    assert n > 0 and n % 256 == 0
    assert L.esc_convattn_workspace_bytes(64, 16, 64, 64, 13) >= 64 * 16 * 9 * 4
    for bad in [(0, 16, 8, 8, 13), (1, 0, 8, 8, 13), (1, 16, 0, 8, 13), (1, 16, 8, 8, 12), (1, 16, 8, 8, 19), (1, 16, 8, 8, 1), (1, 16, 8, 8, -3)]:
        assert L.esc_convattn_workspace_bytes(*bad) == 0


def test_host_side_rejections_launch_nothing(L):
    """Fake, never dereferenced addresses: every call must fail on the host checks."""
    X, O, Wl, Wd, Bd, WS = 0x10000000, 0x20000000, 0x30000000, 0x30100000, 0x30200000, 0x40000000
    big = 1 << 20

    def fwd(x=X, B=1, C=64, Ca=16, H=32, W=32, K=13, wl=Wl, wd=Wd, bd=Bd, out=O, dt=1, lay=1, ws=WS, wsb=big):
        return L.esc_convattn_forward_ex(x, B, C, Ca, H, W, K, wl, wd, bd, out, dt, lay, ws, wsb, None)

    assert fwd(x=None) == 1 and fwd(out=None) == 1 and fwd(wl=None) == 1 and fwd(wd=None) == 1 and fwd(bd=None) == 1
    assert fwd(B=0) == 2 and fwd(H=-3) == 2 and fwd(Ca=0) == 2 and fwd(Ca=65) == 2 and fwd(K=12) == 2 and fwd(K=0) == 2
    assert fwd(K=1) == 2 and fwd(K=-1) == 2   # a 1x1 large kernel cannot hold the 3x3 dynamic kernel it is merged with
    assert fwd(K=19) == 3 and fwd(dt=2) == 3 and fwd(lay=5) == 3
    assert fwd(x=X + 8) == 4 and fwd(out=O + 4) == 4 and fwd(wl=Wl + 1) == 4
    assert fwd(out=X) == 5 and fwd(out=X + 64 * 32 * 32 * 2 - 16) == 5 and fwd(x=O + 16, out=O) == 5
    assert fwd(ws=None) == 6 and fwd(ws=WS + 64) == 6 and fwd(wsb=128) == 6
    # the fixed-signature entry and the stage hooks share the checks
    assert L.esc_convattn_forward(None, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, O, None) == 1
    assert L.esc_convattn_forward(X, 1, 64, 16, 8, 8, 14, Wl, Wd, Bd, O, None) == 2
    assert L.esc_convattn_forward(X, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, X, None) == 5
    assert L.esc_convattn_dynkernel(X, 1, 64, 16, 8, 8, Wd, Bd, None, 0, 0, WS, big, None) == 1
    assert L.esc_convattn_dynkernel(X, 1, 64, 16, 8, 8, Wd, Bd, O, 0, 0, WS, 16, None) == 6
    assert L.esc_convattn_stencil(X, 1, 64, 16, 8, 8, 13, Wl, None, O, 0, 0, None, 0, None) == 1
    assert L.esc_convattn_stencil(X, 1, 64, 16, 8, 8, 13, Wl, Wd, X + 16, 0, 0, None, 0, None) == 5
    assert L.esc_convattn_forward_host(None, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, O, 0, 0) == 1
    assert L.esc_convattn_forward_host(X, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, O, 7, 0) == 3
    # two-layer estimator: the same checks plus the hidden width
    Wu, Bu = 0x30300000, 0x30400000

    def mlp(x=X, wd=Wd, bd=Bd, wu=Wu, bu=Bu, h=8, out=O, ws=WS, wsb=big, K=13):
        return L.esc_convattn_forward_mlp(x, 1, 64, 16, 32, 32, K, Wl, wd, bd, wu, bu, h, out, 1, 1, ws, wsb, None)

    assert mlp(h=0) == 2 and mlp(h=-4) == 2 and mlp(h=129) == 2 and mlp(K=12) == 2
    assert mlp(wd=None) == 1 and mlp(bd=None) == 1 and mlp(wu=None) == 1 and mlp(bu=None) == 1 and mlp(x=None) == 1
    assert mlp(wu=Wu + 1) == 4 and mlp(out=X) == 5 and mlp(wsb=64) == 6
    assert L.esc_convattn_dynkernel_mlp(X, 1, 64, 16, 8, 8, Wd, Bd, Wu, Bu, 0, O, 0, 0, WS, big, None) == 2
    assert L.esc_convattn_dynkernel_mlp(X, 1, 64, 16, 8, 8, Wd, Bd, Wu, Bu, 8, None, 0, 0, WS, big, None) == 1
    assert L.esc_convattn_set_tile_width(48) == 3 and L.esc_convattn_set_tile_width(0) == 0
    # decomposed large kernel: the point-wise filter is one more checked pointer
    Wp = 0x30500000

    def pw(x=X, wp=Wp, out=O, K=13, ws=WS, wsb=big):
        return L.esc_convattn_forward_pw(x, 1, 64, 16, 32, 32, K, Wl, wp, Wd, Bd, out, 1, 1, ws, wsb, None)

    assert pw(wp=None) == 1 and pw(x=None) == 1 and pw(K=14) == 2 and pw(wp=Wp + 1) == 4 and pw(out=X) == 5 and pw(wsb=8) == 6
    assert L.esc_convattn_stencil_pw(X, 1, 64, 16, 8, 8, 13, Wl, None, Wd, O, 0, 0, None, 0, None) == 1
    assert L.esc_convattn_stencil_pw(X, 1, 64, 16, 8, 8, 13, Wl, Wp, Wd, X + 16, 0, 0, None, 0, None) == 5
    Wdn = 0x30600000
    assert L.esc_convattn_forward_dense(X, 1, 64, 16, 32, 32, 13, None, Wd, Bd, O, 1, 1, WS, big, None) == 1
    assert L.esc_convattn_forward_dense(X, 1, 64, 16, 32, 32, 13, Wdn + 1, Wd, Bd, O, 1, 1, WS, big, None) == 4
    assert L.esc_convattn_forward_dense(X, 1, 64, 16, 32, 32, 13, Wdn, Wd, Bd, X, 1, 1, WS, big, None) == 5
    assert L.esc_convattn_stencil_dense(X, 1, 64, 16, 8, 8, 12, Wdn, Wd, O, 0, 0, None, 0, None) == 2
    assert L.esc_convattn_forward_variant(X, 1, 64, 16, 32, 32, 13, 9, Wl, None, None, None, Wd, Bd, 0, O, 1, 1, WS, big, None) == 3
    assert L.esc_convattn_forward_variant(X, 1, 64, 16, 32, 32, 13, 1, Wl, None, None, None, Wd, Bd, 0, O, 1, 1, WS, big, None) == 1
    assert L.esc_convattn_forward_variant(X, 1, 64, 16, 32, 32, 13, 0, Wl, None, None, None, Wd, Bd, 8, O, 1, 1, WS, big, None) == 1
    assert L.esc_convattn_forward_variant(X, 1, 64, 16, 32, 32, 13, 0, Wl, None, None, None, Wd, Bd, -1, O, 1, 1, WS, big, None) == 2
    GO, GX = 0x50000000, 0x60000000
    assert L.esc_convattn_backward(X, GO, 1, 64, 16, 32, 32, 13, Wl, Wd, Bd, None, None, None, None, 1, 1, WS, big, None) == 1
    assert L.esc_convattn_backward(X, GO, 1, 64, 16, 32, 32, 9, Wl, Wd, Bd, GX, None, None, None, 1, 1, WS, big, None) == 3
    assert L.esc_convattn_backward(X, GO, 1, 64, 16, 32, 32, 13, Wl, Wd, Bd, X, None, None, None, 1, 1, WS, big, None) == 5
    assert L.esc_convattn_backward(X, GO, 1, 64, 16, 32, 32, 13, Wl, Wd, Bd, GO + 32, None, None, None, 1, 1, WS, big, None) == 5
    assert L.esc_convattn_backward(X, GO, 1, 64, 16, 32, 32, 13, Wl, Wd, Bd, GX, None, None, None, 1, 1, WS, 64, None) == 6
    assert L.esc_convattn_forward_host_submit(2, X, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, O, 0, 0) == 3
    assert L.esc_convattn_forward_host_submit(0, None, 1, 64, 16, 8, 8, 13, Wl, Wd, Bd, O, 0, 0) == 1
    assert L.esc_convattn_forward_host_wait(-1) == 3
    assert L.esc_convattn_workspace_init(None, 1024, None) == 6
    assert L.esc_convattn_device_status(None, None) == 6


def test_backward_entries_reject_on_the_host(L):
    """Both backward entries check shapes, pointers and the workspace before anything could be launched (fake addresses)."""
    X, GO, GX, Wl, Wa, Wb, Wc, Wd, WS = (0x10000000, 0x18000000, 0x20000000, 0x30000000, 0x30100000, 0x30200000, 0x30300000,
                                         0x30400000, 0x40000000)
    L.esc_convattn_backward_workspace_bytes.restype = ctypes.c_size_t
    need = L.esc_convattn_backward_workspace_bytes(1, 16, 32, 32, 13)
    assert need > 0 and need % 256 == 0
    assert L.esc_convattn_backward_workspace_bytes(1, 16, 32, 32, 9) > 0           # odd K up to 13
    for K in (15, 17, 12, 1):
        assert L.esc_convattn_backward_workspace_bytes(1, 16, 32, 32, K) == 0

    def bwd(x=X, go=GO, K=13, gx=GX, ws=WS, wsb=None, C=64, Ca=16):
        return L.esc_convattn_backward(x, go, 1, C, Ca, 32, 32, K, Wl, Wa, Wb, gx, None, None, None, 1, 1, ws, need if wsb is None else wsb, None)

    def bwd_mlp(hidden=8, gx=GX, K=13, wd=Wa, wsb=None):
        return L.esc_convattn_backward_mlp(X, GO, 1, 64, 16, 32, 32, K, Wl, wd, Wb, Wc, Wd, hidden, gx, None, None, None, None, None, 1, 1,
                                           WS, need if wsb is None else wsb, None)

    assert bwd(K=15) == 3 and bwd(K=12) == 2                                        # unsupported size; even size
    assert bwd(x=None) == 1 and bwd(go=None) == 1 and bwd(gx=None) == 1             # null tensors
    assert bwd(gx=X) == 5                                                           # grad_x over x
    assert bwd(ws=None) == 6 and bwd(wsb=need - 256) == 6 and bwd(ws=WS + 8) == 6   # workspace missing, short, misaligned
    assert bwd(Ca=80) == 2                                                          # C_a > C
    assert bwd_mlp(hidden=0) == 2 and bwd_mlp(hidden=-3) == 2 and bwd_mlp(hidden=129) == 2
    assert bwd_mlp(wd=None) == 1 and bwd_mlp(gx=X) == 5 and bwd_mlp(K=15) == 3 and bwd_mlp(wsb=0) == 6


def test_other_backward_entries_reject_on_the_host(L):
    """The decomposed, dense, any-form and Conv_fuse backward entries: the same checks, before anything could be launched."""
    X, GO, GX, Wl, Wp, Wa, Wb, Wc, Wd, WS = (0x10000000, 0x18000000, 0x20000000, 0x30000000, 0x30100000, 0x30200000, 0x30300000,
                                             0x30400000, 0x30500000, 0x40000000)
    for f in (L.esc_convattn_backward_workspace_bytes, L.esc_convattn_backward_dense_workspace_bytes, L.esc_conv_fuse_backward_workspace_bytes):
        f.restype = ctypes.c_size_t
    need = L.esc_convattn_backward_workspace_bytes(1, 16, 32, 32, 13)
    need_d = L.esc_convattn_backward_dense_workspace_bytes(1, 16, 32, 32, 13)
    assert need_d > need and need_d % 256 == 0
    assert L.esc_convattn_backward_dense_workspace_bytes(1, 8, 32, 32, 13) == 0     # the dense kernel is 16 x 16 channels
    assert L.esc_convattn_backward_dense_workspace_bytes(1, 16, 32, 32, 15) == 0

    def pw(wp=Wp, Ca=16, C=64, gx=GX, wsb=need, K=13):
        return L.esc_convattn_backward_pw(X, GO, 1, C, Ca, 32, 32, K, Wl, wp, Wa, Wb, gx, None, None, None, None, 1, 1, WS, wsb, None)

    assert pw(wp=None) == 1 and pw(Ca=12, C=48) == 3 and pw(gx=GO) == 5 and pw(wsb=256) == 6 and pw(K=15) == 3

    def dense(Ca=16, gx=GX, wsb=need_d, go=GO):
        return L.esc_convattn_backward_dense(X, go, 1, 64, Ca, 32, 32, 13, Wl, Wa, Wb, gx, None, None, None, 1, 1, WS, wsb, None)

    assert dense(Ca=8) == 3 and dense(gx=X) == 5 and dense(go=None) == 1
    assert dense(wsb=need) == 6                                                     # the depth-wise workspace is too small for it

    def variant(form, wp=Wp, hidden=8, wsb=need_d, wdown=Wc):
        return L.esc_convattn_backward_variant(X, GO, 1, 64, 16, 32, 32, 13, form, Wl, wp, wdown, Wd, Wa, Wb, hidden, GX,
                                               None, None, None, None, None, None, 1, 1, WS, wsb, None)

    assert variant(7) == 3 and variant(1, wp=None) == 1 and variant(0, hidden=-1) == 2 and variant(0, hidden=200) == 2
    assert variant(0, wdown=None) == 1 and variant(2, wsb=need) == 6 and variant(0, wsb=0) == 6

    need_f = L.esc_conv_fuse_backward_workspace_bytes(1, 64, 32, 32)
    assert need_f > 0 and need_f % 256 == 0 and L.esc_conv_fuse_backward_workspace_bytes(1, 40, 32, 32) == 0

    def fuse(C=64, cat=X, go=GO, gc=GX, w=Wl, ws=WS, wsb=need_f):
        return L.esc_conv_fuse_backward(cat, go, 1, C, 32, 32, w, gc, None, None, 1, 1, ws, wsb, None)

    assert fuse(C=40) == 3 and fuse(cat=None) == 1 and fuse(w=None) == 1 and fuse(gc=GO) == 5 and fuse(gc=X) == 5
    assert fuse(ws=None) == 6 and fuse(wsb=need_f - 256) == 6 and fuse(go=GO + 2) == 4


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2503_06671_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(RuntimeError, match="no CPU implementation"):
        binding.lib()


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2503_06671_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "synth.py", f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_2503_06671_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f
