"""Single-kernel timings of the NVFP4 library (CUDA events), for tuning and for profiler captures.

  python -m paper_2505_19115_b200.microbench gemm --m 8192 --n 8192 --k 4096 [--tile-n 256] [--bf16-out]
  python -m paper_2505_19115_b200.microbench quantize --rows 16384 --cols 16384 [--transposed] [--sr] [--fp32]
  python -m paper_2505_19115_b200.microbench amax --rows 16384 --cols 16384

  python -m paper_2505_19115_b200.microbench mma_peak [--stages 2048]
      the tensor pipe's issue rate for the GEMM's instruction, no loads: FLOP/clk/SM and TFLOP/s at the clock held
  python -m paper_2505_19115_b200.microbench gemm_account --m 4096 --n 4096 --k 4096
      builds the library with the GEMM's per-role cycle account compiled in and prints where each role of CTA pair 0
      spent its cycles (shares of the role's total)

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




def mma_peak(stages=2048, iters=5, warmup=2, instr_n=256):
    """Issue rate of the block-scaled FP4 MMA on resident operands (see nvfp4_microbench_mma_peak)."""
    MMA_FLOP = 2.0 * 256 * instr_n * 64      # one tcgen05.mma cta_group::2 kind::mxf4nvf4 instruction
    best_ms, out = None, None
    for i in range(warmup + iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = nb.nvfp4_microbench_mma_peak(stages, instr_n)
        e1.record()
        torch.cuda.synchronize()
        if i >= warmup:
            ms = e0.elapsed_time(e1)
            best_ms = ms if best_ms is None else min(best_ms, ms)
    h = out.cpu()
    if int(h[:, 2].max()) != 0:
        raise RuntimeError("mma_peak: a bounded wait ran out")
    cycles = h[:, 0].double()
    pairs, instr = h.shape[0], int(h[0, 1])
    per_instr = float(cycles.median()) / instr
    flop_clk_sm = MMA_FLOP / per_instr / 2.0
    sms = 2 * pairs
    return {"kernel": "mma_peak", "instr_n": instr_n, "pairs": pairs, "instructions_per_pair": instr,
            "cycles_per_instruction_median": per_instr, "cycles_per_instruction_max": float(cycles.max()) / instr,
            "FLOP_per_clk_per_SM": flop_clk_sm, "ms": best_ms,
            "TFLOP/s": pairs * instr * MMA_FLOP / (best_ms * 1e-3) / 1e12,
            "implied_sm_mhz": pairs * instr * MMA_FLOP / (best_ms * 1e-3) / (flop_clk_sm * sms) / 1e6}


def gemm_account(m, n, k, bf16_out=False):
    """Where the roles of CTA pair 0 spend their cycles in one GEMM launch (debug build of the library)."""
    import ctypes as C
    from . import build
    L = C.CDLL(build.build_account())
    vp, i64, ci = C.c_void_p, C.c_int64, C.c_int
    L.nvfp4_gemm.restype = ci
    L.nvfp4_gemm.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, vp, ci, i64, vp]
    L.nvfp4_debug_gemm_account.restype = ci
    L.nvfp4_debug_gemm_account.argtypes = [C.POINTER(C.c_longlong)]
    dev = torch.device("cuda", torch.cuda.current_device())
    A = synth.normal((m, k), 1.0, 1, device=dev)
    B = synth.normal((n, k), 0.02, 2, device=dev)
    ga, gb = nb.nvfp4_tensor_amax_scale(A), nb.nvfp4_tensor_amax_scale(B)
    ac, asf = nb.nvfp4_quantize(A, global_scale=ga, sf_layout=nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(B, global_scale=gb, sf_layout=nb.SF_SWIZZLED)
    out = torch.empty((m, n), dtype=torch.bfloat16 if bf16_out else torch.float32, device=dev)

    def run():
        st = L.nvfp4_gemm(ac.data_ptr(), asf.data_ptr(), ga.data_ptr(), bc.data_ptr(), bsf.data_ptr(), gb.data_ptr(),
                          m, n, k, out.data_ptr(), nb.BF16 if bf16_out else nb.FP32, n, torch.cuda.current_stream().cuda_stream)
        assert st == 0
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    acc = (C.c_longlong * 32)()
    assert L.nvfp4_debug_gemm_account(acc) == 0
    a = list(acc)
    tiles = ((m + 255) // 256) * ((n + 255) // 256)
    pairs = torch.cuda.get_device_properties(dev).multi_processor_count // 2
    tiles_pair0 = len(range(0, tiles, pairs))
    stages = tiles_pair0 * ((k + 255) // 256)

    def share(x, total):
        return round(x / total, 4) if total else None
    return {"kernel": "gemm_account", "m": m, "n": n, "k": k, "out": str(out.dtype), "ms": ms,
            "TFLOP/s": 2.0 * m * n * k / ms / 1e9, "tiles_of_pair0": tiles_pair0, "k_stages_of_pair0": stages,
            "issuer": {"cycles": a[7], "cycles_per_k_stage": a[7] / stages, "wait_accumulator": share(a[4], a[7]),
                       "wait_operands": share(a[5], a[7]), "wait_scales": share(a[6], a[7]),
                       "issuing": share(a[7] - a[4] - a[5] - a[6], a[7])},
            "operand_producer": {"cycles": a[1], "wait_free_stage": share(a[0], a[1])},
            "scale_mover": {"cycles": a[10], "wait_tiles_landed": share(a[8], a[10]), "wait_free_buffer": share(a[9], a[10])},
            "epilogue_warp": {"cycles": a[14], "wait_tile_done": share(a[12], a[14]), "reading_accumulator": share(a[13], a[14]),
                              "accumulator_read_cycles_per_tile": a[13] / tiles_pair0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["gemm", "gemm_bf16", "transpose", "quantize", "dual", "amax", "mma_peak", "gemm_account"])
    ap.add_argument("--stages", type=int, default=2048)
    ap.add_argument("--instr-n", type=int, default=256)
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

    if a.kernel == "mma_peak":
        res = mma_peak(a.stages, a.iters, a.warmup, a.instr_n)
    elif a.kernel == "gemm_account":
        res = gemm_account(a.m, a.n, a.k, a.bf16_out)
    elif a.kernel == "gemm":
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
