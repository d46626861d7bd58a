"""Single-kernel timings of the NVFP4 library (CUDA events), for tuning and for profiler captures.

  python -m paper_2505_19115_b200.microbench gemm --m 8192 --n 8192 --k 4096 [--tile-n 256] [--bf16-out]
  python -m paper_2505_19115_b200.microbench quantize --rows 16384 --cols 16384 [--transposed] [--sr] [--fp32]
  python -m paper_2505_19115_b200.microbench amax --rows 16384 --cols 16384

Prints one JSON line per run: time per launch, TFLOP/s or GB/s (algorithmic bytes).
"""
import argparse
import json

import torch

from . import binding as nb
from . import synth


def _time(fn, iters, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["gemm", "gemm_bf16", "transpose", "quantize", "dual", "amax"])
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--rows", type=int, default=16384)
    ap.add_argument("--cols", type=int, default=16384)
    ap.add_argument("--tile-n", type=int, default=0)
    ap.add_argument("--bf16-out", action="store_true")
    ap.add_argument("--transposed", action="store_true")
    ap.add_argument("--sr", action="store_true")
    ap.add_argument("--fp32", action="store_true")
    ap.add_argument("--linear-sf", action="store_true")
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)

    if a.kernel == "gemm":
        A = synth.normal((a.m, a.k), 1.0, 1, device=dev)
        B = synth.normal((a.n, a.k), 0.02, 2, device=dev)
        ga, gb = nb.nvfp4_tensor_amax_scale(A), nb.nvfp4_tensor_amax_scale(B)
        ac, asf = nb.nvfp4_quantize(A, global_scale=ga, sf_layout=nb.SF_SWIZZLED)
        bc, bsf = nb.nvfp4_quantize(B, global_scale=gb, sf_layout=nb.SF_SWIZZLED)
        del A, B
        out = torch.empty((a.m, a.n), dtype=torch.bfloat16 if a.bf16_out else torch.float32, device=dev)
        nb.nvfp4_gemm_set_tile_n(a.tile_n)
        ms = _time(lambda: nb.nvfp4_gemm(ac, asf, ga, bc, bsf, gb, out=out), a.iters, a.warmup)
        flops = 2.0 * a.m * a.n * a.k
        res = {"kernel": "gemm", "m": a.m, "n": a.n, "k": a.k, "tile_n": a.tile_n, "out": str(out.dtype),
               "ms": ms, "TFLOP/s": flops / ms / 1e9}
    elif a.kernel == "gemm_bf16":
        A = synth.normal((a.m, a.k), 1.0, 1, device=dev)
        B = synth.normal((a.n, a.k), 0.02, 2, device=dev)
        out = torch.empty((a.m, a.n), dtype=torch.bfloat16 if a.bf16_out else torch.float32, device=dev)
        ms = _time(lambda: nb.nvfp4_gemm_bf16(A, B, out=out), a.iters, a.warmup)
        res = {"kernel": "gemm_bf16", "m": a.m, "n": a.n, "k": a.k, "out": str(out.dtype), "ms": ms,
               "TFLOP/s": 2.0 * a.m * a.n * a.k / ms / 1e9}
    elif a.kernel == "transpose":
        x = synth.normal((a.rows, a.cols), 1.0, 3, device=dev)
        ms = _time(lambda: nb.nvfp4_transpose_bf16(x), a.iters, a.warmup)
        res = {"kernel": "transpose", "rows": a.rows, "cols": a.cols, "ms": ms, "GB/s": a.rows * a.cols * 4 / ms / 1e6}
    elif a.kernel == "quantize":
        dt = torch.float32 if a.fp32 else torch.bfloat16
        x = synth.heavy_tailed((a.rows, a.cols), 1002, device=dev, dtype=dt)
        g = nb.nvfp4_tensor_amax_scale(x)
        Rq, Kq = (a.cols, a.rows) if a.transposed else (a.rows, a.cols)
        layout = nb.SF_LINEAR if a.linear_sf else nb.SF_SWIZZLED
        codes = torch.empty((Rq, Kq // 2), dtype=torch.uint8, device=dev)
        sf = torch.empty(nb.nvfp4_sf_bytes(Rq, Kq, layout), dtype=torch.uint8, device=dev)
        r = nb.Rounding(nb.SR, 1, 0) if a.sr else nb.Rounding()
        ms = _time(lambda: nb.nvfp4_quantize(x, a.transposed, g, r, layout, codes=codes, scales=sf), a.iters, a.warmup)
        nbytes = a.rows * a.cols * (x.element_size() + 0.5625)
        res = {"kernel": "quantize", "rows": a.rows, "cols": a.cols, "transposed": a.transposed, "sr": a.sr,
               "dtype": str(dt), "ms": ms, "GB/s": nbytes / ms / 1e6}
    elif a.kernel == "dual":
        x = synth.heavy_tailed((a.rows, a.cols), 1002, device=dev)
        g = nb.nvfp4_tensor_amax_scale(x)
        r = nb.Rounding(nb.SR, 1, 0) if a.sr else nb.Rounding()
        r2 = nb.Rounding(nb.SR, 1, 1) if a.sr else nb.Rounding()
        L = nb.lib()
        cr, sr_, ct, st_ = nb.nvfp4_quantize_dual(x, g, r, r2, nb.SF_SWIZZLED)

        def run():
            import ctypes as C
            s = L.nvfp4_quantize_dual(x.data_ptr(), 0, a.rows, a.cols, x.stride(0), g.data_ptr(), C.byref(r), cr.data_ptr(),
                                      sr_.data_ptr(), C.byref(r2), ct.data_ptr(), st_.data_ptr(), nb.SF_SWIZZLED,
                                      torch.cuda.current_stream().cuda_stream)
            assert s == 0
        ms = _time(run, a.iters, a.warmup)
        res = {"kernel": "dual", "rows": a.rows, "cols": a.cols, "sr": a.sr, "ms": ms,
               "GB/s": a.rows * a.cols * 3.125 / ms / 1e6}
    else:
        x = synth.normal((a.rows, a.cols), 1.0, 3, device=dev)
        out = torch.empty(1, dtype=torch.float32, device=dev)
        ms = _time(lambda: nb.nvfp4_tensor_amax_scale(x, out=out), a.iters, a.warmup)
        res = {"kernel": "amax", "rows": a.rows, "cols": a.cols, "ms": ms, "GB/s": a.rows * a.cols * 2 / ms / 1e6}
    torch.cuda.synchronize()
    res["device_error_word"] = nb.nvfp4_device_error_word()
    print(json.dumps(res))


if __name__ == "__main__":
    main()
