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
