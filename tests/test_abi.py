"""The C-ABI library loads, exports every symbol the header declares, and rejects bad
arguments on the host before touching a device (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2505_19115_b200 import binding as nb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "nvfp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nvfp4_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert {"nvfp4_quantize", "nvfp4_gemm", "nvfp4_linear_fwd", "nvfp4_linear_bwd_dx",
            "nvfp4_linear_bwd_dw"} <= set(names)
    lib = C.CDLL(nb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    assert nb.status_string(0) == "ok"
    for s in range(1, 8):
        assert nb.status_string(s) not in ("ok", "unknown status")
    assert nb.status_string(99) == "unknown status"


def test_sf_bytes():
    assert nb.nvfp4_sf_bytes(128, 64, nb.SF_SWIZZLED) == 512
    assert nb.nvfp4_sf_bytes(129, 80, nb.SF_SWIZZLED) == 2 * 2 * 512
    assert nb.nvfp4_sf_bytes(3, 48, nb.SF_LINEAR) == 9
    assert nb.nvfp4_sf_bytes(3, 40, nb.SF_LINEAR) == 0
    assert nb.nvfp4_sf_bytes(3, 48, 7) == 0


def test_workspace_bytes():
    for which in (0, 1, 2):
        n = nb.nvfp4_linear_workspace_bytes(256, 512, 512, which)
        assert n > 0 and n % 256 == 0
    assert nb.nvfp4_linear_workspace_bytes(256, 512, 512, 5) == 0
    assert nb.nvfp4_linear_workspace_bytes(0, 512, 512, 0) == 0
    # the size query refuses exactly the layers the calls refuse: a contraction length that is a multiple
    # of 16 but not of 32 (K for fwd, N for dx, M for dw), or a contiguous axis that is not a multiple of 8
    assert nb.nvfp4_linear_workspace_bytes(256, 512, 528, 0) == 0
    assert nb.nvfp4_linear_workspace_bytes(256, 528, 512, 1) == 0
    assert nb.nvfp4_linear_workspace_bytes(272, 512, 512, 2) == 0
    assert nb.nvfp4_linear_workspace_bytes(256, 516, 512, 0) == 0          # Y rows of 516 elements
    assert nb.nvfp4_linear_workspace_bytes(256, 512, 544, 0) > 0


def test_static_forward_rejects_what_the_size_query_rejects():
    L = nb.lib()
    r = nb.Rounding()
    buf = C.c_void_p(0x1000)
    st = L.nvfp4_linear_fwd_static(buf, buf, 0, 256, 512, 528, 0, None, None, C.byref(r), C.byref(r), buf, 1, None)
    assert st == 2                                                          # shape error, not a late failure


def test_quantize_argument_errors_are_host_side():
    L = nb.lib()
    r = nb.Rounding()
    buf = C.c_void_p(0x1000)          # never dereferenced: every call below fails validation first
    q = lambda **kw: L.nvfp4_quantize(
        kw.get("x", buf), kw.get("dtype", 0), kw.get("rows", 16), kw.get("cols", 32), kw.get("ld", 32),
        kw.get("transposed", 0), None, kw.get("r", C.byref(r)), kw.get("codes", buf), kw.get("scales", buf),
        kw.get("sf", 0), None)
    assert q(x=None) == 1 and q(codes=None) == 1 and q(scales=None) == 1 and q(r=None) == 1
    assert q(dtype=3) == 4 and q(sf=2) == 4 and q(transposed=2) == 4
    assert q(r=C.byref(nb.Rounding(5))) == 4
    assert q(cols=24, ld=24) == 2 and q(rows=0) == 2 and q(ld=16) == 2
    assert q(rows=24, transposed=1) == 2
    assert q(x=C.c_void_p(0x1008)) == 3 and q(ld=36) == 3
    assert L.nvfp4_tensor_amax_scale(None, 0, 1, 8, 8, buf, None) == 1
    assert L.nvfp4_tensor_amax_scale(buf, 0, 1, 12, 12, buf, None) == 2


def test_gemm_and_linear_argument_errors_are_host_side():
    L = nb.lib()
    buf = C.c_void_p(0x1000)
    g = lambda **kw: L.nvfp4_gemm(kw.get("a", buf), buf, None, buf, buf, None, kw.get("M", 128), kw.get("N", 128),
                                  kw.get("K", 256), kw.get("d", buf), kw.get("dt", 1), kw.get("ldd", 128), None)
    assert g(a=None) == 1 and g(d=None) == 1
    assert g(K=24) == 2 and g(M=0) == 2 and g(ldd=64) == 2
    assert g(dt=9) == 4
    assert g(d=C.c_void_p(0x1004)) == 3 and g(ldd=130) == 3
    r = nb.Rounding()
    lin = lambda fn, **kw: fn(kw.get("a", buf), buf, 0, kw.get("M", 256), kw.get("N", 512), kw.get("K", 512), kw.get("gm", 0),
                              None, None, C.byref(r), C.byref(r), buf, 1, kw.get("ws", buf), kw.get("wsb", 1 << 30), None)
    for fn in (L.nvfp4_linear_fwd, L.nvfp4_linear_bwd_dx, L.nvfp4_linear_bwd_dw):
        assert lin(fn, a=None) == 1
        assert lin(fn, ws=None) == 5 and lin(fn, wsb=16) == 5
        assert lin(fn, gm=7) == 4
        assert lin(fn, gm=2) == 1          # G_GIVEN without scale pointers
    # the contraction axis (K, N, M respectively) must be a multiple of 32
    assert lin(L.nvfp4_linear_fwd, K=528) == 2
    assert lin(L.nvfp4_linear_bwd_dx, N=528) == 2
    assert lin(L.nvfp4_linear_bwd_dw, M=272) == 2


def test_newer_entry_points_reject_bad_arguments_on_the_host():
    L = nb.lib()
    r = nb.Rounding()
    rb = C.byref(r)
    buf = C.c_void_p(0x1000)
    # both orientations from one read
    d = lambda **kw: L.nvfp4_quantize_dual(kw.get("x", buf), kw.get("dtype", 0), kw.get("rows", 32), kw.get("cols", 32),
                                           kw.get("ld", 32), None, kw.get("rr", rb), buf, buf, rb, kw.get("ct", buf), buf,
                                           kw.get("sf", 0), None)
    assert d(x=None) == 1 and d(ct=None) == 1 and d(rr=None) == 1
    assert d(rows=24) == 2 and d(cols=24, ld=24) == 2 and d(ld=16) == 2
    assert d(dtype=2) == 4 and d(sf=3) == 4
    assert d(x=C.c_void_p(0x1004)) == 3
    # fused layer calls: sizes and workspace
    assert nb.nvfp4_linear_saved_bytes(256, 512, 512) % 256 == 0 and nb.nvfp4_linear_saved_bytes(256, 512, 500) == 0
    for which in (0, 1, 2):
        assert nb.nvfp4_linear_fused_workspace_bytes(256, 512, 512, which) > 0
    assert nb.nvfp4_linear_fused_workspace_bytes(256, 512, 512, 3) == 0
    fs = lambda **kw: L.nvfp4_linear_fwd_save(kw.get("X", buf), buf, 0, kw.get("M", 256), 512, 512, kw.get("gm", 0), None, None,
                                              rb, rb, rb, rb, buf, 1, kw.get("sv", buf), kw.get("svb", 1 << 30), buf, 1 << 30, None)
    assert fs(X=None) == 1 and fs(M=250) == 2 and fs(gm=5) == 4 and fs(sv=None) == 5 and fs(svb=64) == 5 and fs(gm=2) == 1
    bs = lambda **kw: L.nvfp4_linear_bwd_saved(kw.get("dY", buf), 0, 256, kw.get("N", 512), 512, 0, None, rb, rb, buf, 1 << 30,
                                               buf, 1, buf, kw.get("dwt", 1), kw.get("ws", buf), 1 << 30, None)
    assert bs(dY=None) == 1 and bs(N=500) == 2 and bs(dwt=7) == 4 and bs(ws=None) == 5
    # chained layers: quantized output / quantized input
    qo = lambda **kw: L.nvfp4_linear_fwd_qout(kw.get("X", buf), buf, 0, 256, kw.get("N", 512), kw.get("K", 512), kw.get("gm", 0), None, None,
                                              rb, rb, None, kw.get("ry", rb), kw.get("yc", buf), buf, kw.get("sf", 1),
                                              kw.get("ws", buf), 1 << 30, None)
    assert qo(X=None) == 1 and qo(ry=None) == 1 and qo(yc=None) == 1 and qo(N=528) == 2 and qo(K=528) == 2
    assert qo(gm=9) == 4 and qo(gm=2) == 1 and qo(ws=None) == 5 and qo(sf=5) == 4
    qi = lambda **kw: L.nvfp4_linear_fwd_qin(kw.get("xc", buf), buf, None, kw.get("W", buf), 0, 256, 512, kw.get("K", 512), kw.get("gm", 0),
                                             None, rb, buf, kw.get("yt", 1), kw.get("ws", buf), 1 << 30, None)
    assert qi(xc=None) == 1 and qi(W=None) == 1 and qi(K=528) == 2 and qi(gm=9) == 4 and qi(gm=2) == 1
    assert qi(yt=3) == 4 and qi(ws=None) == 5
    # quantized epilogue, bf16 and MXFP4 products, noise monitor, transpose
    gq = lambda **kw: L.nvfp4_gemm_quantized(kw.get("a", buf), buf, None, buf, buf, None, 128, kw.get("N", 128), 256, None,
                                             kw.get("r", rb), buf, buf, kw.get("sf", 0), None)
    assert gq(a=None) == 1 and gq(r=None) == 1 and gq(N=144) == 2 and gq(sf=9) == 4
    gb = lambda **kw: L.nvfp4_gemm_bf16(kw.get("a", buf), buf, 128, 128, kw.get("K", 64), buf, kw.get("dt", 1), kw.get("ldd", 128), None)
    assert gb(a=None) == 1 and gb(K=24) == 2 and gb(dt=5) == 4 and gb(ldd=130) == 3
    gm = lambda **kw: L.nvfp4_gemm_mx(kw.get("a", buf), buf, None, buf, buf, None, 128, 128, kw.get("K", 256), buf, 1, 128, None)
    assert gm(a=None) == 1 and gm(K=48) == 2
    qm = lambda **kw: L.nvfp4_quantize_mx(kw.get("x", buf), kw.get("dtype", 0), kw.get("rows", 32), kw.get("cols", 64), 64, kw.get("tr", 0), None, rb,
                                          buf, buf, 0, kw.get("ws", None), 0, None)
    assert qm(x=None) == 1 and qm(cols=48) == 2 and qm(tr=1, dtype=1) == 4
    assert qm(tr=1, rows=1 << 25) == 5          # beyond the tile kernel's grid: needs the transpose workspace
    assert nb.nvfp4_sf_bytes_mx(128, 128, nb.SF_SWIZZLED) == 512 and nb.nvfp4_sf_bytes_mx(3, 64, nb.SF_LINEAR) == 6
    assert nb.nvfp4_sf_bytes_mx(3, 48, nb.SF_LINEAR) == 0
    nz = lambda **kw: L.nvfp4_quantization_noise(kw.get("x", buf), 0, 32, kw.get("cols", 32), 32, 0, None, buf, buf, 0,
                                                 kw.get("sums", buf), None)
    assert nz(x=None) == 1 and nz(sums=None) == 1 and nz(cols=24) == 2 and nz(sums=C.c_void_p(0x1004)) == 3
    tr = lambda **kw: L.nvfp4_transpose_bf16(kw.get("x", buf), kw.get("rows", 64), 64, 64, buf, None)
    assert tr(x=None) == 1 and tr(rows=60) == 2
    assert L.nvfp4_linear_bwd_bf16_workspace_bytes(256, 512, 512) == 0          # operands are read in place
    gx = lambda **kw: L.nvfp4_gemm_bf16_ex(kw.get("a", buf), kw.get("am", 0), buf, kw.get("bm", 0), kw.get("M", 128), 128, 64, buf, 1, 128, None)
    assert gx(a=None) == 1 and gx(am=2) == 4 and gx(am=1, bm=0) == 4 and gx(am=1, bm=1, M=100) == 2
