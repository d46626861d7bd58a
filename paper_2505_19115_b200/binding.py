"""Thin ctypes binding over libnvfp4.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/nvfp4.h).
torch tensors are used for device memory and streams; all computation happens
inside the CUDA library.  There is no CPU fallback: if the library is missing
or a call fails, an exception is raised.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnvfp4.so")

BF16, FP32 = 0, 1
RTN, SR = 0, 1
SF_LINEAR, SF_SWIZZLED = 0, 1
G_NONE, G_AMAX, G_GIVEN = 0, 1, 2
LINEAR_FWD, LINEAR_BWD_DX, LINEAR_BWD_DW = 0, 1, 2


class NvFp4Error(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: nvfp4 status {status} ({status_string(status)})")


class Rounding(C.Structure):
    _fields_ = [("mode", C.c_int32), ("reserved", C.c_int32), ("seed", C.c_uint64), ("offset", C.c_uint64)]

    def __init__(self, mode=RTN, seed=0, offset=0):
        super().__init__(mode, 0, seed, offset)


_lib = None


def lib():
    """Load libnvfp4.so (built in-tree by paper_2505_19115_b200/build.py).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2505_19115_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, ci, sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
    rp = C.POINTER(Rounding)
    L.nvfp4_status_string.restype = C.c_char_p
    L.nvfp4_status_string.argtypes = [ci]
    L.nvfp4_sf_bytes.restype = sz
    L.nvfp4_sf_bytes.argtypes = [i64, i64, ci]
    L.nvfp4_quantize.restype = ci
    L.nvfp4_quantize.argtypes = [vp, ci, i64, i64, i64, ci, vp, rp, vp, vp, ci, vp]
    L.nvfp4_quantize_dual.restype = ci
    L.nvfp4_quantize_dual.argtypes = [vp, ci, i64, i64, i64, vp, rp, vp, vp, rp, vp, vp, ci, vp]
    L.nvfp4_quantization_noise.restype = ci
    L.nvfp4_quantization_noise.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp, ci, vp, vp]
    L.nvfp4_tensor_amax_scale.restype = ci
    L.nvfp4_tensor_amax_scale.argtypes = [vp, ci, i64, i64, i64, vp, vp]
    L.nvfp4_gemm.restype = ci
    L.nvfp4_gemm.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, i64, vp]
    L.nvfp4_gemm_quantized.restype = ci
    L.nvfp4_gemm_quantized.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, rp, vp, vp, ci, vp]
    L.nvfp4_gemm_set_tile_n.restype = ci
    L.nvfp4_gemm_set_tile_n.argtypes = [ci]
    L.nvfp4_linear_workspace_bytes.restype = sz
    L.nvfp4_linear_workspace_bytes.argtypes = [i64, i64, i64, ci]
    lin = [vp, vp, ci, i64, i64, i64, ci, vp, vp, rp, rp, vp, ci, vp, sz, vp]
    for name in ("nvfp4_linear_fwd", "nvfp4_linear_bwd_dx", "nvfp4_linear_bwd_dw"):
        getattr(L, name).restype = ci
        getattr(L, name).argtypes = lin
    L.nvfp4_linear_fwd_qout.restype = ci
    L.nvfp4_linear_fwd_qout.argtypes = [vp, vp, ci, i64, i64, i64, ci, vp, vp, rp, rp, vp, rp, vp, vp, ci, vp, sz, vp]
    L.nvfp4_linear_fwd_qin.restype = ci
    L.nvfp4_linear_fwd_qin.argtypes = [vp, vp, vp, vp, ci, i64, i64, i64, ci, vp, rp, vp, ci, vp, sz, vp]
    L.nvfp4_linear_saved_bytes.restype = sz
    L.nvfp4_linear_saved_bytes.argtypes = [i64, i64, i64]
    L.nvfp4_linear_fused_workspace_bytes.restype = sz
    L.nvfp4_linear_fused_workspace_bytes.argtypes = [i64, i64, i64, ci]
    L.nvfp4_linear_fwd_save.restype = ci
    L.nvfp4_linear_fwd_save.argtypes = [vp, vp, ci, i64, i64, i64, ci, vp, vp, rp, rp, rp, rp, vp, ci, vp, sz, vp, sz, vp]
    L.nvfp4_linear_bwd_saved.restype = ci
    L.nvfp4_linear_bwd_saved.argtypes = [vp, ci, i64, i64, i64, ci, vp, rp, rp, vp, sz, vp, ci, vp, ci, vp, sz, vp]
    L.nvfp4_linear_bwd.restype = ci
    L.nvfp4_linear_bwd.argtypes = [vp, vp, vp, ci, i64, i64, i64, ci, vp, vp, vp, rp, rp, rp, rp, vp, ci, vp, ci, vp, sz, vp]
    L.nvfp4_sf_bytes_mx.restype = sz
    L.nvfp4_sf_bytes_mx.argtypes = [i64, i64, ci]
    L.nvfp4_quantize_mx.restype = ci
    L.nvfp4_quantize_mx.argtypes = [vp, ci, i64, i64, i64, ci, vp, rp, vp, vp, ci, vp, sz, vp]
    L.nvfp4_gemm_mx.restype = ci
    L.nvfp4_gemm_mx.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, i64, vp]
    L.nvfp4_gemm_bf16.restype = ci
    L.nvfp4_gemm_bf16.argtypes = [vp, vp, i64, i64, i64, vp, ci, i64, vp]
    L.nvfp4_gemm_bf16_ex.restype = ci
    L.nvfp4_gemm_bf16_ex.argtypes = [vp, ci, vp, ci, i64, i64, i64, vp, ci, i64, vp]
    L.nvfp4_transpose_bf16.restype = ci
    L.nvfp4_transpose_bf16.argtypes = [vp, i64, i64, i64, vp, vp]
    L.nvfp4_linear_bwd_bf16_workspace_bytes.restype = sz
    L.nvfp4_linear_bwd_bf16_workspace_bytes.argtypes = [i64, i64, i64]
    L.nvfp4_linear_bwd_bf16.restype = ci
    L.nvfp4_linear_bwd_bf16.argtypes = [vp, vp, vp, i64, i64, i64, vp, ci, vp, ci, vp, sz, vp]
    L.nvfp4_linear_fwd_static.restype = ci
    L.nvfp4_linear_fwd_static.argtypes = [vp, vp, ci, i64, i64, i64, ci, vp, vp, rp, rp, vp, ci, vp]
    L.nvfp4_microbench_mma_peak.restype = ci
    L.nvfp4_microbench_mma_peak.argtypes = [ci, ci, vp, sz, C.POINTER(C.c_int), vp]
    L.nvfp4_device_error_word.restype = ci
    L.nvfp4_device_error_word.argtypes = [C.POINTER(C.c_uint32)]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().nvfp4_status_string(status).decode()


def _check(status, where):
    if status != 0:
        raise NvFp4Error(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def nvfp4_sf_bytes(Rq: int, Kq: int, sf_layout: int = SF_SWIZZLED) -> int:
    return int(lib().nvfp4_sf_bytes(Rq, Kq, sf_layout))


def nvfp4_quantize(x: torch.Tensor, transposed: bool = False, global_scale: torch.Tensor = None,
                   rounding: Rounding = None, sf_layout: int = SF_LINEAR, codes: torch.Tensor = None,
                   scales: torch.Tensor = None, stream=None):
    """Returns (codes [Rq, Kq/2] u8, scales u8: [Rq, Kq/16] linear or a flat swizzled buffer)."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    Rq, Kq = (cols, rows) if transposed else (rows, cols)
    rounding = rounding or Rounding()
    if codes is None:
        codes = torch.empty((Rq, max(Kq // 2, 1)), dtype=torch.uint8, device=x.device)
    if scales is None:
        if sf_layout == SF_LINEAR:
            scales = torch.empty((Rq, max(Kq // 16, 1)), dtype=torch.uint8, device=x.device)
        else:
            scales = torch.empty(max(nvfp4_sf_bytes(Rq, Kq, sf_layout), 16), dtype=torch.uint8, device=x.device)
    st = lib().nvfp4_quantize(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), int(transposed),
                              _ptr(global_scale), C.byref(rounding), _ptr(codes), _ptr(scales), sf_layout,
                              _stream(stream))
    _check(st, "nvfp4_quantize")
    return codes, scales


def nvfp4_quantize_dual(x: torch.Tensor, global_scale: torch.Tensor = None, rounding_row: Rounding = None,
                        rounding_t: Rounding = None, sf_layout: int = SF_LINEAR, stream=None):
    """Row and transposed quantization from one read.  Returns (codes_row, scales_row, codes_t, scales_t)."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    rounding_row = rounding_row or Rounding()
    rounding_t = rounding_t or Rounding()

    def bufs(Rq, Kq):
        codes = torch.empty((Rq, max(Kq // 2, 1)), dtype=torch.uint8, device=x.device)
        if sf_layout == SF_LINEAR:
            return codes, torch.empty((Rq, max(Kq // 16, 1)), dtype=torch.uint8, device=x.device)
        return codes, torch.empty(max(nvfp4_sf_bytes(Rq, Kq, sf_layout), 16), dtype=torch.uint8, device=x.device)

    cr, sr = bufs(rows, cols)
    ct, stt = bufs(cols, rows)
    st = lib().nvfp4_quantize_dual(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), _ptr(global_scale),
                                   C.byref(rounding_row), _ptr(cr), _ptr(sr), C.byref(rounding_t), _ptr(ct), _ptr(stt),
                                   sf_layout, _stream(stream))
    _check(st, "nvfp4_quantize_dual")
    return cr, sr, ct, stt


def nvfp4_quantization_noise(x: torch.Tensor, codes, scales, transposed: bool = False, global_scale=None,
                             sf_layout: int = SF_LINEAR, stream=None) -> torch.Tensor:
    """Device tensor of two doubles: sum (Q(x) - x)^2 and sum x^2 (Section 4's noise and norm)."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    sums = torch.empty(2, dtype=torch.float64, device=x.device)
    st = lib().nvfp4_quantization_noise(_ptr(x), _dtype_code(x), x.shape[0], x.shape[1], x.stride(0), int(transposed),
                                        _ptr(global_scale), _ptr(codes), _ptr(scales), sf_layout, _ptr(sums),
                                        _stream(stream))
    _check(st, "nvfp4_quantization_noise")
    return sums


def nvfp4_tensor_amax_scale(x: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=x.device)
    st = lib().nvfp4_tensor_amax_scale(_ptr(x), _dtype_code(x), x.shape[0], x.shape[1], x.stride(0), _ptr(out),
                                       _stream(stream))
    _check(st, "nvfp4_tensor_amax_scale")
    return out


def nvfp4_gemm(a_codes, a_sf, a_g, b_codes, b_sf, b_g, out_dtype=torch.float32, out: torch.Tensor = None,
               stream=None) -> torch.Tensor:
    """D[M,N] = A[M,K] . B[N,K]^T on packed codes with swizzled scales."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a_codes.device)
    st = lib().nvfp4_gemm(_ptr(a_codes), _ptr(a_sf), _ptr(a_g), _ptr(b_codes), _ptr(b_sf), _ptr(b_g),
                          M, N, K, _ptr(out), _dtype_code(out), out.stride(0), _stream(stream))
    _check(st, "nvfp4_gemm")
    return out


def nvfp4_gemm_quantized(a_codes, a_sf, a_g, b_codes, b_sf, b_g, out_global_scale=None, rounding: Rounding = None,
                         sf_layout: int = SF_LINEAR, stream=None):
    """Q(A . B^T) with blocks along N, straight from the GEMM epilogue.  Returns (codes [M, N/2], scales)."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    rounding = rounding or Rounding()
    codes = torch.empty((M, N // 2), dtype=torch.uint8, device=a_codes.device)
    if sf_layout == SF_LINEAR:
        scales = torch.empty((M, N // 16), dtype=torch.uint8, device=a_codes.device)
    else:
        scales = torch.empty(max(nvfp4_sf_bytes(M, N, sf_layout), 16), dtype=torch.uint8, device=a_codes.device)
    st = lib().nvfp4_gemm_quantized(_ptr(a_codes), _ptr(a_sf), _ptr(a_g), _ptr(b_codes), _ptr(b_sf), _ptr(b_g), M, N, K,
                                    _ptr(out_global_scale), C.byref(rounding), _ptr(codes), _ptr(scales), sf_layout,
                                    _stream(stream))
    _check(st, "nvfp4_gemm_quantized")
    return codes, scales


def nvfp4_gemm_set_tile_n(bn: int) -> None:
    _check(lib().nvfp4_gemm_set_tile_n(bn), "nvfp4_gemm_set_tile_n")


def nvfp4_linear_workspace_bytes(M: int, N: int, K: int, which: int) -> int:
    return int(lib().nvfp4_linear_workspace_bytes(M, N, K, which))


def _linear(name, which, a, b, M, N, K, out_shape, gscale_mode, ga, gb, ra, rb, out, out_dtype, workspace, stream):
    if out is None:
        out = torch.empty(out_shape, dtype=out_dtype, device=a.device)
    if workspace is None:
        workspace = torch.empty(nvfp4_linear_workspace_bytes(M, N, K, which), dtype=torch.uint8, device=a.device)
    assert a.is_contiguous() and b.is_contiguous() and out.is_contiguous() and a.dtype == b.dtype
    st = getattr(lib(), name)(_ptr(a), _ptr(b), _dtype_code(a), M, N, K, gscale_mode, _ptr(ga), _ptr(gb),
                              C.byref(ra), C.byref(rb), _ptr(out), _dtype_code(out), _ptr(workspace),
                              workspace.numel(), _stream(stream))
    _check(st, name)
    return out


def nvfp4_linear_fwd(X, W, gscale_mode=G_AMAX, gx=None, gw=None, rx=None, rw=None, out=None,
                     out_dtype=torch.float32, workspace=None, stream=None):
    """Y[M,N] = Q(X) . Q(W)^T (Eq. 1/4).  Default rounding: RtN for both."""
    (M, K), N = X.shape, W.shape[0]
    return _linear("nvfp4_linear_fwd", LINEAR_FWD, X, W, M, N, K, (M, N), gscale_mode, gx, gw,
                   rx or Rounding(RTN), rw or Rounding(RTN), out, out_dtype, workspace, stream)


def nvfp4_linear_bwd_dx(dY, W, gscale_mode=G_AMAX, gdy=None, gw=None, rdy=None, rw=None, out=None,
                        out_dtype=torch.float32, workspace=None, stream=None):
    """dX[M,K] = Q(dY) . Q(W^T)^T (Eq. 2/5).  Default rounding: SR for dY, RtN for W^T."""
    (M, N), K = dY.shape, W.shape[1]
    return _linear("nvfp4_linear_bwd_dx", LINEAR_BWD_DX, dY, W, M, N, K, (M, K), gscale_mode, gdy, gw,
                   rdy or Rounding(SR, 0, 0), rw or Rounding(RTN), out, out_dtype, workspace, stream)


def nvfp4_linear_bwd_dw(dY, X, gscale_mode=G_AMAX, gdy=None, gx=None, rdy=None, rx=None, out=None,
                        out_dtype=torch.float32, workspace=None, stream=None):
    """dW[N,K] = Q(dY^T) . Q(X^T)^T (Eq. 3/6).  Default rounding: SR for both."""
    (M, N), K = dY.shape, X.shape[1]
    return _linear("nvfp4_linear_bwd_dw", LINEAR_BWD_DW, dY, X, M, N, K, (N, K), gscale_mode, gdy, gx,
                   rdy or Rounding(SR, 0, 1), rx or Rounding(SR, 0, 2), out, out_dtype, workspace, stream)


def nvfp4_linear_fwd_qout(X, W, gy=None, ry=None, gscale_mode=G_AMAX, gx=None, gw=None, rx=None, rw=None,
                          sf_layout=SF_SWIZZLED, codes=None, scales=None, workspace=None, stream=None):
    """Forward layer whose output leaves the GEMM already quantized along N: returns (codes [M, N/2], scales)."""
    (M, K), N = X.shape, W.shape[0]
    if codes is None:
        codes = torch.empty((M, N // 2), dtype=torch.uint8, device=X.device)
    if scales is None:
        if sf_layout == SF_LINEAR:
            scales = torch.empty((M, N // 16), dtype=torch.uint8, device=X.device)
        else:
            scales = torch.empty(max(nvfp4_sf_bytes(M, N, sf_layout), 16), dtype=torch.uint8, device=X.device)
    if workspace is None:
        workspace = torch.empty(nvfp4_linear_workspace_bytes(M, N, K, LINEAR_FWD), dtype=torch.uint8, device=X.device)
    assert X.is_contiguous() and W.is_contiguous() and X.dtype == W.dtype
    st = lib().nvfp4_linear_fwd_qout(_ptr(X), _ptr(W), _dtype_code(X), M, N, K, gscale_mode, _ptr(gx), _ptr(gw),
                                     C.byref(rx or Rounding(RTN)), C.byref(rw or Rounding(RTN)), _ptr(gy),
                                     C.byref(ry or Rounding(RTN)), _ptr(codes), _ptr(scales), sf_layout,
                                     _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "nvfp4_linear_fwd_qout")
    return codes, scales


def nvfp4_linear_fwd_qin(x_codes, x_scales, gx, W, gscale_mode=G_AMAX, gw=None, rw=None, out=None,
                         out_dtype=torch.float32, workspace=None, stream=None):
    """Forward layer for an input already quantized along K (codes [M, K/2], swizzled scales, per-tensor scale gx)."""
    M, K = x_codes.shape[0], x_codes.shape[1] * 2
    N = W.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=W.device)
    if workspace is None:
        workspace = torch.empty(nvfp4_linear_workspace_bytes(M, N, K, LINEAR_FWD), dtype=torch.uint8, device=W.device)
    assert W.is_contiguous() and out.is_contiguous()
    st = lib().nvfp4_linear_fwd_qin(_ptr(x_codes), _ptr(x_scales), _ptr(gx), _ptr(W), _dtype_code(W), M, N, K, gscale_mode,
                                    _ptr(gw), C.byref(rw or Rounding(RTN)), _ptr(out), _dtype_code(out), _ptr(workspace),
                                    workspace.numel(), _stream(stream))
    _check(st, "nvfp4_linear_fwd_qin")
    return out


FUSED_FWD_SAVE, FUSED_BWD_SAVED, FUSED_BWD = 0, 1, 2


def nvfp4_linear_saved_bytes(M, N, K) -> int:
    return int(lib().nvfp4_linear_saved_bytes(M, N, K))


def nvfp4_linear_fused_workspace_bytes(M, N, K, which) -> int:
    return int(lib().nvfp4_linear_fused_workspace_bytes(M, N, K, which))


def _scratch(nbytes, device, given):
    if given is not None:
        return given
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def nvfp4_linear_fwd_save(X, W, gscale_mode=G_AMAX, gx=None, gw=None, rx=None, rw=None, rxt=None, rwt=None, out=None,
                          out_dtype=torch.float32, saved=None, workspace=None, stream=None):
    """Y = Q(X) . Q(W)^T and, from the same reads, Q(X^T) and Q(W^T) into `saved` for the backward
    and update passes.  Returns (Y, saved).  Default rounding: the paper's (RtN, RtN, SR for X^T, RtN for W^T)."""
    (M, K), N = X.shape, W.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=X.device)
    saved = _scratch(nvfp4_linear_saved_bytes(M, N, K), X.device, saved)
    ws = _scratch(nvfp4_linear_fused_workspace_bytes(M, N, K, FUSED_FWD_SAVE), X.device, workspace)
    st = lib().nvfp4_linear_fwd_save(_ptr(X), _ptr(W), _dtype_code(X), M, N, K, gscale_mode, _ptr(gx), _ptr(gw),
                                     C.byref(rx or Rounding(RTN)), C.byref(rw or Rounding(RTN)),
                                     C.byref(rxt or Rounding(SR, 0, 2)), C.byref(rwt or Rounding(RTN)),
                                     _ptr(out), _dtype_code(out), _ptr(saved), saved.numel(), _ptr(ws), ws.numel(),
                                     _stream(stream))
    _check(st, "nvfp4_linear_fwd_save")
    return out, saved


def nvfp4_linear_bwd_saved(dY, saved, K, gscale_mode=G_AMAX, gdy=None, rdy=None, rdyt=None, dX=None, dW=None,
                           dx_dtype=torch.float32, dw_dtype=torch.float32, workspace=None, stream=None):
    """dX and dW from one read of dY and the operands nvfp4_linear_fwd_save kept.  Returns (dX, dW)."""
    M, N = dY.shape
    if dX is None:
        dX = torch.empty((M, K), dtype=dx_dtype, device=dY.device)
    if dW is None:
        dW = torch.empty((N, K), dtype=dw_dtype, device=dY.device)
    ws = _scratch(nvfp4_linear_fused_workspace_bytes(M, N, K, FUSED_BWD_SAVED), dY.device, workspace)
    st = lib().nvfp4_linear_bwd_saved(_ptr(dY), _dtype_code(dY), M, N, K, gscale_mode, _ptr(gdy),
                                      C.byref(rdy or Rounding(SR, 0, 0)), C.byref(rdyt or Rounding(SR, 0, 1)),
                                      _ptr(saved), saved.numel(), _ptr(dX), _dtype_code(dX), _ptr(dW), _dtype_code(dW),
                                      _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "nvfp4_linear_bwd_saved")
    return dX, dW


def nvfp4_linear_bwd(dY, W, X, gscale_mode=G_AMAX, gdy=None, gw=None, gx=None, rdy=None, rdyt=None, rwt=None, rxt=None,
                     dX=None, dW=None, dx_dtype=torch.float32, dw_dtype=torch.float32, workspace=None, stream=None):
    """dX and dW (Eq. 2/5 and Eq. 3/6) with dY read once.  Returns (dX, dW)."""
    (M, N), K = dY.shape, W.shape[1]
    if dX is None:
        dX = torch.empty((M, K), dtype=dx_dtype, device=dY.device)
    if dW is None:
        dW = torch.empty((N, K), dtype=dw_dtype, device=dY.device)
    ws = _scratch(nvfp4_linear_fused_workspace_bytes(M, N, K, FUSED_BWD), dY.device, workspace)
    st = lib().nvfp4_linear_bwd(_ptr(dY), _ptr(W), _ptr(X), _dtype_code(dY), M, N, K, gscale_mode, _ptr(gdy), _ptr(gw),
                                _ptr(gx), C.byref(rdy or Rounding(SR, 0, 0)), C.byref(rdyt or Rounding(SR, 0, 1)),
                                C.byref(rwt or Rounding(RTN)), C.byref(rxt or Rounding(SR, 0, 2)),
                                _ptr(dX), _dtype_code(dX), _ptr(dW), _dtype_code(dW), _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "nvfp4_linear_bwd")
    return dX, dW


def nvfp4_sf_bytes_mx(Rq: int, Kq: int, sf_layout: int = SF_SWIZZLED) -> int:
    return int(lib().nvfp4_sf_bytes_mx(Rq, Kq, sf_layout))


def nvfp4_quantize_mx(x, transposed: bool = False, global_scale=None, rounding: Rounding = None,
                      sf_layout: int = SF_LINEAR, stream=None):
    """MXFP4 (blocks of 32, E8M0 scales).  Returns (codes [Rq, Kq/2], scales: [Rq, Kq/32] or a flat swizzled buffer)."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    Rq, Kq = (cols, rows) if transposed else (rows, cols)
    rounding = rounding or Rounding()
    codes = torch.empty((Rq, Kq // 2), dtype=torch.uint8, device=x.device)
    if sf_layout == SF_LINEAR:
        scales = torch.empty((Rq, Kq // 32), dtype=torch.uint8, device=x.device)
    else:
        scales = torch.empty(max(nvfp4_sf_bytes_mx(Rq, Kq, sf_layout), 16), dtype=torch.uint8, device=x.device)
    def call(ws):
        return lib().nvfp4_quantize_mx(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), int(transposed), _ptr(global_scale),
                                       C.byref(rounding), _ptr(codes), _ptr(scales), sf_layout, _ptr(ws),
                                       ws.numel() if ws is not None else 0, _stream(stream))
    st = call(None)
    if st == 5 and transposed:          # a shape the tile kernel does not take: the library transposes into a workspace first
        st = call(torch.empty(rows * cols * 2, dtype=torch.uint8, device=x.device))
    _check(st, "nvfp4_quantize_mx")
    return codes, scales


def nvfp4_gemm_mx(a_codes, a_sf, a_g, b_codes, b_sf, b_g, out_dtype=torch.float32, out=None, stream=None):
    """D[M,N] = A[M,K] . B[N,K]^T on MXFP4 operands with swizzled E8M0 scales."""
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a_codes.device)
    st = lib().nvfp4_gemm_mx(_ptr(a_codes), _ptr(a_sf), _ptr(a_g), _ptr(b_codes), _ptr(b_sf), _ptr(b_g), M, N, K,
                             _ptr(out), _dtype_code(out), out.stride(0), _stream(stream))
    _check(st, "nvfp4_gemm_mx")
    return out


def nvfp4_gemm_bf16(A, B, out_dtype=torch.float32, out=None, stream=None):
    """D[M,N] = A[M,K] . B[N,K]^T on bf16 operands (the QAF phase's backward / update precision)."""
    assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.is_contiguous() and B.is_contiguous()
    (M, K), N = A.shape, B.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    _check(lib().nvfp4_gemm_bf16(_ptr(A), _ptr(B), M, N, K, _ptr(out), _dtype_code(out), out.stride(0), _stream(stream)),
           "nvfp4_gemm_bf16")
    return out


def nvfp4_gemm_bf16_ex(A, a_mn_major, B, b_mn_major, out_dtype=torch.float32, out=None, stream=None):
    """D[M,N] = A . B^T on bf16 operands; an MN-major operand is passed as its stored [K, M] (or [K, N]) array."""
    assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.is_contiguous() and B.is_contiguous()
    (K, M) = A.shape if a_mn_major else A.shape[::-1]
    N = B.shape[1] if b_mn_major else B.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    _check(lib().nvfp4_gemm_bf16_ex(_ptr(A), int(a_mn_major), _ptr(B), int(b_mn_major), M, N, K, _ptr(out), _dtype_code(out),
                                    out.stride(0), _stream(stream)), "nvfp4_gemm_bf16_ex")
    return out


def nvfp4_transpose_bf16(x, stream=None):
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    out = torch.empty((x.shape[1], x.shape[0]), dtype=torch.bfloat16, device=x.device)
    _check(lib().nvfp4_transpose_bf16(_ptr(x), x.shape[0], x.shape[1], x.stride(0), _ptr(out), _stream(stream)),
           "nvfp4_transpose_bf16")
    return out


def nvfp4_linear_bwd_bf16(dY, W, X, dx_dtype=torch.float32, dw_dtype=torch.float32, workspace=None, stream=None):
    """QAF backward + update in BF16: returns (dX[M,K], dW[N,K])."""
    (M, N), K = dY.shape, W.shape[1]
    dX = torch.empty((M, K), dtype=dx_dtype, device=dY.device)
    dW = torch.empty((N, K), dtype=dw_dtype, device=dY.device)
    ws = _scratch(int(lib().nvfp4_linear_bwd_bf16_workspace_bytes(M, N, K)), dY.device, workspace)
    _check(lib().nvfp4_linear_bwd_bf16(_ptr(dY), _ptr(W), _ptr(X), M, N, K, _ptr(dX), _dtype_code(dX), _ptr(dW),
                                       _dtype_code(dW), _ptr(ws), ws.numel(), _stream(stream)), "nvfp4_linear_bwd_bf16")
    return dX, dW


STATIC_WORKSPACE_BYTES = 8 << 20


def nvfp4_linear_fwd_static(X, W, gscale_mode=G_AMAX, gx=None, gw=None, rx=None, rw=None, out=None,
                            out_dtype=torch.float32, stream=None):
    """nvfp4_linear_fwd for callers that cannot allocate or pass scratch memory (for instance when
    the whole device already belongs to the host framework's pool): the scratch is a fixed
    STATIC_WORKSPACE_BYTES array inside the library, shared by all calls on a device, so calls
    that may overlap on the GPU must be serialised.  Larger layers raise (status 5)."""
    (M, K), N = X.shape, W.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=X.device)
    rx, rw = rx or Rounding(RTN), rw or Rounding(RTN)
    assert X.is_contiguous() and W.is_contiguous() and out.is_contiguous() and X.dtype == W.dtype
    st = lib().nvfp4_linear_fwd_static(_ptr(X), _ptr(W), _dtype_code(X), M, N, K, gscale_mode, _ptr(gx), _ptr(gw),
                                       C.byref(rx), C.byref(rw), _ptr(out), _dtype_code(out), _stream(stream))
    _check(st, "nvfp4_linear_fwd_static")
    return out


def nvfp4_microbench_mma_peak(stages: int, instr_n: int = 256, device=None, stream=None) -> torch.Tensor:
    """Issue-rate measurement of the FP4 tensor-core instruction: returns an int64 tensor [pairs, 3] of
    (cycles, instructions, timed-out flag) per CTA pair."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    out = torch.zeros((torch.cuda.get_device_properties(dev).multi_processor_count // 2 + 1, 3), dtype=torch.int64, device=dev)
    pairs = C.c_int(0)
    _check(lib().nvfp4_microbench_mma_peak(stages, instr_n, _ptr(out), out.numel() * 8, C.byref(pairs), _stream(stream)),
           "nvfp4_microbench_mma_peak")
    return out[:pairs.value]


def nvfp4_device_error_word() -> int:
    w = C.c_uint32(0)
    _check(lib().nvfp4_device_error_word(C.byref(w)), "nvfp4_device_error_word")
    return int(w.value)
