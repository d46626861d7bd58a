"""ctypes access to the CPU oracle (test infrastructure, never used by the product).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this module.  Arrays are numpy, host memory; nothing here touches CUDA.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_lib = None

_u8p = np.ctypeslib.ndpointer(dtype=np.uint8, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(dtype=np.uint16, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(dtype=np.int64, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(dtype=np.uint32, flags="C_CONTIGUOUS")


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.nvfp4o_e2m1_decode.restype = C.c_float
        L.nvfp4o_e2m1_decode.argtypes = [C.c_uint8]
        L.nvfp4o_e4m3_encode.restype = C.c_uint8
        L.nvfp4o_e4m3_encode.argtypes = [C.c_float]
        L.nvfp4o_e4m3_decode.restype = C.c_float
        L.nvfp4o_e4m3_decode.argtypes = [C.c_uint8]
        L.nvfp4o_philox4x32_10.restype = None
        L.nvfp4o_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
        L.nvfp4o_block_random_u16.restype = None
        L.nvfp4o_block_random_u16.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, _u16p]
        L.nvfp4o_word_random_u16.restype = None
        L.nvfp4o_word_random_u16.argtypes = [C.c_uint32, _u16p]
        L.nvfp4o_round_rtn.restype = C.c_uint8
        L.nvfp4o_round_rtn.argtypes = [C.c_float]
        L.nvfp4o_round_sr.restype = C.c_uint8
        L.nvfp4o_round_sr.argtypes = [C.c_float, C.c_uint16]
        L.nvfp4o_round_sr_many.restype = None
        L.nvfp4o_round_sr_many.argtypes = [C.c_float, _u16p, C.c_int64, _u8p]
        q = [_f32p, C.c_int64, C.c_int64, C.c_float, C.c_int, C.c_uint64, C.c_uint64, _u8p, _u8p, C.c_int]
        L.nvfp4o_quantize.restype = None
        L.nvfp4o_quantize.argtypes = q
        L.nvfp4o_quantize_rows.restype = None
        L.nvfp4o_quantize_rows.argtypes = q[:7] + [C.c_int64] + q[7:]
        L.nvfp4o_quantize_transposed.restype = None
        L.nvfp4o_quantize_transposed.argtypes = q
        L.nvfp4o_dequantize.restype = None
        L.nvfp4o_e8m0_encode_up.restype = C.c_uint8
        L.nvfp4o_e8m0_encode_up.argtypes = [C.c_float]
        L.nvfp4o_e8m0_decode.restype = C.c_float
        L.nvfp4o_e8m0_decode.argtypes = [C.c_uint8]
        L.nvfp4o_quantize_mx_rows.restype = None
        L.nvfp4o_quantize_mx_rows.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_float, C.c_int, C.c_uint64, C.c_uint64,
                                              C.c_int64, _u8p, _u8p, C.c_int]
        L.nvfp4o_dequantize_mx.restype = None
        L.nvfp4o_dequantize_mx.argtypes = [_u8p, _u8p, C.c_float, C.c_int64, C.c_int64, _f32p]
        L.nvfp4o_gemm_mx.restype = None
        L.nvfp4o_gemm_mx.argtypes = [_u8p, _u8p, C.c_float, _u8p, _u8p, C.c_float, C.c_int64, C.c_int64, C.c_int64,
                                     _f32p, _f32p, C.c_int]
        L.nvfp4o_matmul_nt.restype = None
        L.nvfp4o_matmul_nt.argtypes = [_f32p, _f32p, C.c_int64, C.c_int64, C.c_int64, _f32p, _f32p, C.c_int]
        L.nvfp4o_noise_sums.restype = None
        L.nvfp4o_noise_sums.argtypes = [_f32p, _u8p, _u8p, C.c_float, C.c_int64, C.c_int64,
                                        np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")]
        L.nvfp4o_dequantize.argtypes = [_u8p, _u8p, C.c_float, C.c_int64, C.c_int64, _f32p]
        L.nvfp4o_tensor_amax_scale.restype = C.c_float
        L.nvfp4o_tensor_amax_scale.argtypes = [_f32p, C.c_int64]
        g = [_u8p, _u8p, C.c_float, _u8p, _u8p, C.c_float, C.c_int64, C.c_int64, C.c_int64]
        L.nvfp4o_gemm.restype = None
        L.nvfp4o_gemm.argtypes = g + [C.c_void_p, C.c_void_p, C.c_int]
        L.nvfp4o_gemm_f32acc.restype = None
        L.nvfp4o_gemm_f32acc.argtypes = g + [_f32p, C.c_int]
        L.nvfp4o_gemm_sampled.restype = None
        L.nvfp4o_gemm_sampled.argtypes = g + [_i64p, _i64p, C.c_int64, _f32p, _f32p, C.c_int]
        L.nvfp4o_sf_swizzled_offset.restype = C.c_int64
        L.nvfp4o_sf_swizzled_offset.argtypes = [C.c_int64, C.c_int64, C.c_int64]
        L.nvfp4o_sf_swizzled_bytes.restype = C.c_int64
        L.nvfp4o_sf_swizzled_bytes.argtypes = [C.c_int64, C.c_int64]
        L.nvfp4o_sf_swizzle.restype = None
        L.nvfp4o_sf_swizzle.argtypes = [_u8p, C.c_int64, C.c_int64, _u8p]
        _lib = L
    return _lib


RTN, SR = 0, 1


def host_threads() -> int:
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def _f32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def e2m1_decode(code: int) -> float:
    return float(lib().nvfp4o_e2m1_decode(code))


def e4m3_encode(v: float) -> int:
    return int(lib().nvfp4o_e4m3_encode(float(np.float32(v))))


def e4m3_decode(code: int) -> float:
    return float(lib().nvfp4o_e4m3_decode(code))


def philox4x32_10(key, ctr):
    out = np.zeros(4, dtype=np.uint32)
    lib().nvfp4o_philox4x32_10(np.asarray(key, dtype=np.uint32), np.asarray(ctr, dtype=np.uint32), out)
    return out


def block_random_u16(seed: int, offset: int, block: int):
    out = np.zeros(16, dtype=np.uint16)
    lib().nvfp4o_block_random_u16(seed, offset, block, out)
    return out


def word_random_u16(word: int):
    out = np.zeros(4, dtype=np.uint16)
    lib().nvfp4o_word_random_u16(word, out)
    return out


def round_rtn(y: float) -> int:
    return int(lib().nvfp4o_round_rtn(float(np.float32(y))))


def round_sr(y: float, r16: int) -> int:
    return int(lib().nvfp4o_round_sr(float(np.float32(y)), r16))


def round_sr_many(y: float, r16) -> np.ndarray:
    r16 = np.ascontiguousarray(r16, dtype=np.uint16)
    out = np.zeros(r16.size, dtype=np.uint8)
    lib().nvfp4o_round_sr_many(float(np.float32(y)), r16, r16.size, out)
    return out


def quantize(x, g=1.0, mode=RTN, seed=0, offset=0, transposed=False, nthreads=None):
    """x: 2-D array (values already representable in the source dtype, widened
    to fp32).  Returns (codes [Rq, Kq/2] u8, scales [Rq, Kq/16] u8)."""
    x = _f32(x)
    rows, cols = x.shape
    Rq, Kq = (cols, rows) if transposed else (rows, cols)
    assert Kq % 16 == 0
    codes = np.zeros((Rq, Kq // 2), dtype=np.uint8)
    scales = np.zeros((Rq, Kq // 16), dtype=np.uint8)
    nt = host_threads() if nthreads is None else nthreads
    fn = lib().nvfp4o_quantize_transposed if transposed else lib().nvfp4o_quantize
    fn(x, rows, cols, float(np.float32(g)), mode, seed, offset, codes, scales, nt)
    return codes, scales


def quantize_rows(x, first_row, g=1.0, mode=RTN, seed=0, offset=0, nthreads=None):
    """Row quantization of a slice x = full[first_row : first_row + x.shape[0]] of a taller tensor
    (for a transposed quantization pass the transposed slice of columns and the first column)."""
    x = _f32(x)
    rows, cols = x.shape
    assert cols % 16 == 0
    codes = np.zeros((rows, cols // 2), dtype=np.uint8)
    scales = np.zeros((rows, cols // 16), dtype=np.uint8)
    nt = host_threads() if nthreads is None else nthreads
    lib().nvfp4o_quantize_rows(x, rows, cols, float(np.float32(g)), mode, seed, offset, first_row, codes, scales, nt)
    return codes, scales


def dequantize(codes, scales, g=1.0):
    Rq, half = codes.shape
    out = np.zeros((Rq, half * 2), dtype=np.float32)
    lib().nvfp4o_dequantize(np.ascontiguousarray(codes), np.ascontiguousarray(scales),
                            float(np.float32(g)), Rq, half * 2, out)
    return out


def noise_sums(x, codes, scales, g=1.0):
    """(sum (Q(x)-x)^2, sum x^2) in double; x in the quantized orientation [Rq, Kq]."""
    x = _f32(x)
    out = np.zeros(2, dtype=np.float64)
    lib().nvfp4o_noise_sums(x, np.ascontiguousarray(codes), np.ascontiguousarray(scales), float(np.float32(g)),
                            x.shape[0], x.shape[1], out)
    return float(out[0]), float(out[1])


def e8m0_encode_up(v: float) -> int:
    return int(lib().nvfp4o_e8m0_encode_up(float(np.float32(v))))


def e8m0_decode(code: int) -> float:
    return float(lib().nvfp4o_e8m0_decode(code))


def quantize_mx(x, g=1.0, mode=RTN, seed=0, offset=0, transposed=False, first_row=0, nthreads=None):
    """MXFP4: blocks of 32 along the quantized rows, E8M0 scales.  Returns (codes [Rq, Kq/2], scales [Rq, Kq/32]).
    transposed: quantize the transpose of x (blocks along x's rows)."""
    x = _f32(x)
    if transposed:
        x = np.ascontiguousarray(x.T)
    Rq, Kq = x.shape
    assert Kq % 32 == 0
    codes = np.zeros((Rq, Kq // 2), dtype=np.uint8)
    scales = np.zeros((Rq, Kq // 32), dtype=np.uint8)
    lib().nvfp4o_quantize_mx_rows(x, Rq, Kq, float(np.float32(g)), mode, seed, offset, first_row, codes, scales,
                                  host_threads() if nthreads is None else nthreads)
    return codes, scales


def dequantize_mx(codes, scales, g=1.0):
    Rq, half = codes.shape
    out = np.zeros((Rq, half * 2), dtype=np.float32)
    lib().nvfp4o_dequantize_mx(np.ascontiguousarray(codes), np.ascontiguousarray(scales), float(np.float32(g)), Rq,
                               half * 2, out)
    return out


def gemm_mx(a_codes, a_sf, ga, b_codes, b_sf, gb, nthreads=None):
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    D = np.zeros((M, N), dtype=np.float32)
    T = np.zeros((M, N), dtype=np.float32)
    lib().nvfp4o_gemm_mx(np.ascontiguousarray(a_codes), np.ascontiguousarray(a_sf), float(np.float32(ga)),
                         np.ascontiguousarray(b_codes), np.ascontiguousarray(b_sf), float(np.float32(gb)), M, N, K, D, T,
                         host_threads() if nthreads is None else nthreads)
    return D, T


def matmul_nt(A, B, nthreads=None):
    """(A . B^T rounded to fp32 from a double accumulation, sum |a b|) for plain fp32 arrays A[M,K], B[N,K]."""
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    N = B.shape[0]
    D = np.zeros((M, N), dtype=np.float32)
    T = np.zeros((M, N), dtype=np.float32)
    lib().nvfp4o_matmul_nt(A, B, M, N, K, D, T, host_threads() if nthreads is None else nthreads)
    return D, T


def tensor_amax_scale(x) -> float:
    x = _f32(x).reshape(-1)
    return float(lib().nvfp4o_tensor_amax_scale(x, x.size))


def gemm(a_codes, a_sf, ga, b_codes, b_sf, gb, want_T=True, nthreads=None):
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    D = np.zeros((M, N), dtype=np.float32)
    T = np.zeros((M, N), dtype=np.float32) if want_T else None
    nt = host_threads() if nthreads is None else nthreads
    lib().nvfp4o_gemm(np.ascontiguousarray(a_codes), np.ascontiguousarray(a_sf), float(np.float32(ga)),
                      np.ascontiguousarray(b_codes), np.ascontiguousarray(b_sf), float(np.float32(gb)),
                      M, N, K, D.ctypes.data, T.ctypes.data if want_T else None, nt)
    return (D, T) if want_T else D


def gemm_f32acc(a_codes, a_sf, ga, b_codes, b_sf, gb, nthreads=None):
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    D = np.zeros((M, N), dtype=np.float32)
    nt = host_threads() if nthreads is None else nthreads
    lib().nvfp4o_gemm_f32acc(np.ascontiguousarray(a_codes), np.ascontiguousarray(a_sf), float(np.float32(ga)),
                             np.ascontiguousarray(b_codes), np.ascontiguousarray(b_sf), float(np.float32(gb)),
                             M, N, K, D, nt)
    return D


def gemm_sampled(a_codes, a_sf, ga, b_codes, b_sf, gb, ii, jj, nthreads=None):
    M, K = a_codes.shape[0], a_codes.shape[1] * 2
    N = b_codes.shape[0]
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    D = np.zeros(ii.size, dtype=np.float32)
    T = np.zeros(ii.size, dtype=np.float32)
    lib().nvfp4o_gemm_sampled(np.ascontiguousarray(a_codes), np.ascontiguousarray(a_sf), float(np.float32(ga)),
                              np.ascontiguousarray(b_codes), np.ascontiguousarray(b_sf), float(np.float32(gb)),
                              M, N, K, ii, jj, ii.size, D, T, host_threads() if nthreads is None else nthreads)
    return D, T


def sf_swizzled_offset(r, kb, n_kb) -> int:
    return int(lib().nvfp4o_sf_swizzled_offset(r, kb, n_kb))


def sf_swizzled_bytes(Rq, n_kb) -> int:
    return int(lib().nvfp4o_sf_swizzled_bytes(Rq, n_kb))


def sf_swizzle(linear):
    linear = np.ascontiguousarray(linear, dtype=np.uint8)
    Rq, n_kb = linear.shape
    out = np.zeros(sf_swizzled_bytes(Rq, n_kb), dtype=np.uint8)
    lib().nvfp4o_sf_swizzle(linear, Rq, n_kb, out)
    return out
