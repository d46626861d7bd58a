#!/usr/bin/env python
"""Benchmark of the NVFP4 quantize-then-GEMM hot path on B200.

One "step" is one pass of the whole hot path over one Llama-7B-shaped transformer block's five
linear layers (tokens 16384, hidden 4096): for each layer the forward product (Eq. 1/4), the
input-gradient product (Eq. 2/5) and the weight-gradient product (Eq. 3/6), each with its
per-tensor amax passes, its operand quantizations and its block-scaled GEMM, all through the C-ABI
layer calls nvfp4_linear_fwd_save / nvfp4_linear_bwd_saved.

Prints ONE JSON line (rank 0).  Beside the headline it carries: the GEMM's roofline record (every
GEMM launch of the workload bracketed by CUDA events, against the measured peaks and against the
tensor pipe's own issue rate measured in the same run), the quantizer bandwidths, the other
workload configurations (350M block, 65536-token weight gradient, delayed per-tensor scales, bf16
outputs, quantization fused into the producing GEMM), the end-to-end figure with host buffers and
the CPU oracle timed on the host cores.  `--impl reference` times the CPU oracle on a bounded
sample of the same workload instead.
"""
import argparse
import ctypes as C
import json
import os
import statistics
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_19115_b200 import replicas, synth  # noqa: E402

METRIC = "NVFP4 linear fwd+bwd TFLOPS (% FP4 peak); quantizer GB/s (% HBM peak)"
FP4_OVER_BF16 = 4.0        # nominal dense ratio: 9 PFLOP/s NVFP4 vs 2.25 PFLOP/s bf16
NOMINAL_FP4_TFLOPS = 9000.0
MMA_FLOP_PER_CLK_PER_SM = 32768.0   # 2 * 256 * 256 * 64 FLOP per 128 cycles on a CTA pair (microbench mma_peak measures it)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic of the GEMM kernel from the committed ncu capture (profiles/gemm2_nvfp4_kernel_8192x8192x4096.md):
# 82.9 MB read + 211.2 MB written for 306.2 MB of algorithmic bytes (operand codes and scales + fp32 output).
# GEMM traffic follows bytes, not FLOPs, so the workload's figure is this ratio times its own algorithmic bytes.
GEMM_TRAFFIC_RATIO = (82.91 + 211.22) / 306.2


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def block_flops(cfg):
    return sum(6.0 * cfg["tokens"] * K * N for _, K, N in cfg["linears"])


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock, power and the clock-event reasons of one GPU through NVML from a host
    thread (every 10 ms unless told otherwise) while a timed region runs."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, device_index, interval_s=0.01):
        self.idx = device_index
        self.interval_s = interval_s
        self.thread = None
        self.stop_flag = False
        self.sm, self.power, self.mask = [], [], 0
        self.smax = None
        self.error = None

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.idx
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if self.idx < len(ids) and ids[self.idx].isdigit():
                    idx = int(ids[self.idx])
            h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.smax = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self.stop_flag:
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                try:
                    self.power.append(pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0)
                    self.mask |= int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                except Exception:
                    pass
                time.sleep(self.interval_s)
        except Exception as e:  # the number is still reported, without a clock record
            self.error = repr(e)

    def start(self):
        import threading
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()
        return self

    def mark(self):
        """Drops what was sampled so far (warm-up), so the record covers the timed region only."""
        self.sm, self.power, self.mask = [], [], 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.smax, "reasons": [], "samples": 0}
        if self.thread is None:
            return out
        self.stop_flag = True
        self.thread.join(timeout=5)
        if self.sm:
            out.update(sm_mhz=statistics.median(self.sm), sm_min_mhz=min(self.sm), sm_max_mhz=self.smax,
                       reasons=[n for n, bit in self.REASONS if self.mask & bit], samples=len(self.sm))
            if self.power:
                out["power_w_max"] = max(self.power)
        if self.error:
            out["error"] = self.error
        return out


# ------------------------------------------------------------------------------------------------
# the CPU oracle on the host cores (a reported baseline, not a target)
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(cfg, rows=256, seed=2004, nthreads=None):
    """One bounded sample of the workload on the host: the first layer's forward product for the
    first `rows` tokens (quantize those rows of X, quantize all of W, dequantize-then-matmul)."""
    from oracle import binding as ob
    name, K, N = cfg["linears"][0]
    X = synth.normal((rows, K), 1.0, seed, device="cpu").float().numpy()
    W = synth.normal((N, K), 0.02, seed + 1, device="cpu").float().numpy()
    t0 = time.perf_counter()
    gx, gw = ob.tensor_amax_scale(X), ob.tensor_amax_scale(W)
    xc, xs = ob.quantize(X, g=gx, nthreads=nthreads)
    wc, ws = ob.quantize(W, g=gw, nthreads=nthreads)
    ob.gemm(xc, xs, gx, wc, ws, gw, want_T=False, nthreads=nthreads)
    dt = time.perf_counter() - t0
    flops = 2.0 * rows * K * N
    return flops, dt, f"layer '{name}' forward product on the first {rows} of {cfg['tokens']} tokens " \
                      f"(quantize X rows + all of W, dequantize-then-matmul in double)"


def cpu_baseline_record(cfg):
    """The oracle as it stands on the host cores: the forward-product slice at all cores and at one thread
    (with the linear extrapolation to the whole block step labelled as such) and its quantizer on a whole
    2^24-element tensor in GB/s at both thread counts.  About 20-30 s of CPU work."""
    from oracle import binding as ob
    cores = ob.host_threads()
    f_all, s_all, sample = oracle_sample_step(cfg, rows=256)
    f_one, s_one, _ = oracle_sample_step(cfg, rows=16, nthreads=1)
    tf_all, tf_one = f_all / s_all / 1e12, f_one / s_one / 1e12
    x = synth.heavy_tailed(synth.square_shape(2 ** 24), seed=1001, device="cpu").float().numpy()
    g = ob.tensor_amax_scale(x)
    qbytes = x.size * 2.5625                       # the bf16 source's bytes, as for the GPU figure
    quant = {"elements": int(x.size), "bytes_per_element": 2.5625}
    for label, mode in (("rtn", ob.RTN), ("sr", ob.SR)):
        for tl, nt in (("all_cores", cores), ("1_thread", 1)):
            t0 = time.perf_counter()
            ob.quantize(x, g=g, mode=mode, seed=1, nthreads=nt)
            quant[f"row_{label}_{tl}_GBs"] = qbytes / (time.perf_counter() - t0) / 1e9
    step_flops = block_flops(cfg)
    return {"value": tf_all, "unit": "TFLOPS", "cores": cores, "kind": "oracle",
            "sample": sample + f"; {s_all:.1f} s on {cores} threads",
            "matmul_slice": {"all_cores_TFLOPS": tf_all, "all_cores_rows": 256, "one_thread_TFLOPS": tf_one,
                             "one_thread_rows": 16,
                             "extrapolated_block_step_s_all_cores": step_flops / (tf_all * 1e12),
                             "extrapolated_block_step_s_one_thread": step_flops / (tf_one * 1e12),
                             "extrapolation": "linear in FLOPs from the measured slice (labelled estimate, not a measurement)"},
            "quantizer_2p24": quant}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import binding as ob
    cfg = synth.LLAMA_7B
    rows = 64                                    # about two seconds per step on 16 cores, so that K steps stay within minutes
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample_step(cfg, rows=rows)
    flops = secs = 0.0
    sample = ""
    for _ in range(args.steps):
        f, dt, sample = oracle_sample_step(cfg, rows=rows)
        flops += f
        secs += dt
    val = flops / secs / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "nvfp4 (e2m1 x ue4m3), f64 accumulate",
        "data": "synthetic", "config": {"workload": "llama7b_block_linears_fwd_bwd", "tokens": cfg["tokens"],
                                        "hidden": cfg["hidden"], "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOPS", "cores": ob.host_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------------
class Block:
    """The five linear layers of one transformer block with resident inputs and outputs, and the fused
    layer calls that make one step: forward (Eq. 1/4) keeping Q(X^T), Q(W^T); backward + update
    (Eq. 2/5, 3/6) from one read of dY.  Each tensor's amax is taken once, each tensor read once per pass."""

    def __init__(self, nb, cfg, dev, rank, act_dtype=torch.float32, dw_dtype=torch.float32):
        self.nb, self.cfg, self.M = nb, cfg, cfg["tokens"]
        M = self.M
        self.layers = []
        for li, (name, K, N) in enumerate(cfg["linears"]):
            X, W, dY = synth.linear_inputs(M, K, N, seed=replicas.replica_seed(4000 + 10 * li, rank), device=dev)
            self.layers.append(dict(name=name, K=K, N=N, X=X, W=W, dY=dY,
                                    Y=torch.empty((M, N), dtype=act_dtype, device=dev),
                                    dX=torch.empty((M, K), dtype=act_dtype, device=dev),
                                    dW=torch.empty((N, K), dtype=dw_dtype, device=dev)))
        ws_bytes = max(nb.nvfp4_linear_fused_workspace_bytes(M, l["N"], l["K"], w) for l in self.layers
                       for w in (nb.FUSED_FWD_SAVE, nb.FUSED_BWD_SAVED))
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.saved = torch.empty(max(nb.nvfp4_linear_saved_bytes(M, l["N"], l["K"]) for l in self.layers),
                                 dtype=torch.uint8, device=dev)
        self.rt = nb.Rounding(nb.RTN)
        self.sr = [nb.Rounding(nb.SR, 0, o) for o in range(3)]      # distinct offsets per SR site
        self.in_bytes = sum(t.numel() * t.element_size() for l in self.layers for t in (l["X"], l["W"], l["dY"]))
        self.flops = block_flops(cfg)
        self.given = None

    def compute_given_scales(self):
        """Per-tensor scales computed once, as a training loop with delayed scaling would carry them over."""
        nb = self.nb
        self.given = [{k: nb.nvfp4_tensor_amax_scale(l[k]) for k in ("X", "W", "dY")} for l in self.layers]

    def layer(self, l, gmode, g=None):
        nb, rt, sr = self.nb, self.rt, self.sr
        gx, gw, gdy = (g["X"], g["W"], g["dY"]) if g else (None, None, None)
        nb.nvfp4_linear_fwd_save(l["X"], l["W"], gmode, gx=gx, gw=gw, rx=rt, rw=rt, rxt=sr[2], rwt=rt, out=l["Y"],
                                 saved=self.saved, workspace=self.ws)
        nb.nvfp4_linear_bwd_saved(l["dY"], self.saved, l["K"], gmode, gdy=gdy, rdy=sr[0], rdyt=sr[1], dX=l["dX"],
                                  dW=l["dW"], workspace=self.ws)

    def step(self, gmode=None):
        gmode = self.nb.G_AMAX if gmode is None else gmode
        for i, l in enumerate(self.layers):
            self.layer(l, gmode, self.given[i] if gmode == self.nb.G_GIVEN else None)

    def launches_per_step(self, gmode=None):
        per_layer = 3 + 3 if gmode == self.nb.G_GIVEN else 3 + 3 + 3   # dual quantizers, GEMMs (+ amax sweeps)
        return len(self.layers) * per_layer


def timed_graph(step, steps, barrier, use_graph=True, sampler=None):
    """W warm-up steps are the caller's; captures `step` into a CUDA graph (one replay untimed) and times
    `steps` replays with CUDA events.  Returns (ms_total, launch_mode)."""
    run, mode = step, "stream"
    if use_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            run, mode = graph.replay, "cuda_graph"
        except Exception as e:                  # capture refused: time the plain launches and say so
            mode = f"stream (graph capture failed: {type(e).__name__})"
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler is not None:
        sampler.mark()
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    barrier()
    return e0.elapsed_time(e1), mode


def time_call(fn, reps, warm=3, graph=False):
    """Milliseconds per call (CUDA events).  graph=True replays `reps` calls from one CUDA graph, which keeps the
    host's launch cost (10-20 us per call from Python) out of the figure for kernels that run only a few microseconds."""
    for _ in range(warm):
        fn()
    run, n = fn, reps
    if graph:
        try:
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for _ in range(reps):
                    fn()
            g.replay()
            run, n = g.replay, 1
        except Exception:
            run, n = fn, reps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        run()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def quantizer_sweep(nb, dev, peaks, peak_kind):
    """Quantizer bandwidth on the heavy-tailed tensors: 2^28 elements (exceeds L2: the HBM figure) and, labelled
    as L2-resident and launch-bound, 2^24 and 2^20.  Bytes = 2 + 0.5 + 1/16 per element (3.125 for both orientations)."""
    rt = nb.Rounding(nb.RTN)
    out = {"bytes_per_element": 2.5625, "peak_hbm_gbs": peaks["hbm_gbs"], "peak_kind": peak_kind}
    L = nb.lib()
    for n_el, reps, note in ((2 ** 28, 10, None),
                             (2 ** 24, 30, "L2-resident: 32 MiB of input, not an HBM figure; back-to-back launches replayed from a CUDA graph"),
                             (2 ** 20, 50, "L2-resident and launch-bound: 2 MiB of input, a few microseconds per launch; back-to-back "
                                           "launches replayed from a CUDA graph")):
        small = n_el < 2 ** 28
        xq = synth.heavy_tailed(synth.square_shape(n_el), seed=1002, device=dev)
        R, Cc = xq.shape
        gq = nb.nvfp4_tensor_amax_scale(xq)
        codes = torch.empty((R, Cc // 2), dtype=torch.uint8, device=dev)
        sfs = torch.empty(nb.nvfp4_sf_bytes(R, Cc, nb.SF_SWIZZLED), dtype=torch.uint8, device=dev)
        ct = torch.empty((Cc, R // 2), dtype=torch.uint8, device=dev)
        st = torch.empty(nb.nvfp4_sf_bytes(Cc, R, nb.SF_SWIZZLED), dtype=torch.uint8, device=dev)
        rec = {"elements": n_el}
        if note:
            rec["note"] = note
        for label, tr, rr in (("row_rtn", False, rt), ("row_sr", False, nb.Rounding(nb.SR, 1, 0)),
                              ("transposed_rtn", True, rt), ("transposed_sr", True, nb.Rounding(nb.SR, 1, 0))):
            c_, s_ = (ct, st) if tr else (codes, sfs)
            ms = time_call(lambda: nb.nvfp4_quantize(xq, tr, gq, rr, nb.SF_SWIZZLED, codes=c_, scales=s_), reps, graph=small)
            gbs = n_el * 2.5625 / (ms * 1e-3) / 1e9
            rec[label] = {"GB/s": gbs, "us": ms * 1e3, "frac_of_measured_copy": gbs / peaks["hbm_gbs"], "frac_of_8TBs": gbs / 8000.0}
        # both orientations from one read (the fused layer's quantizer): 2 + 2 * 0.5625 bytes per element
        for label, r1, r2 in (("dual_rtn", rt, rt), ("dual_sr", nb.Rounding(nb.SR, 1, 0), nb.Rounding(nb.SR, 1, 1))):
            def dual():
                stt = L.nvfp4_quantize_dual(xq.data_ptr(), nb.BF16, R, Cc, xq.stride(0), gq.data_ptr(),
                                            C.byref(r1), codes.data_ptr(), sfs.data_ptr(), C.byref(r2), ct.data_ptr(),
                                            st.data_ptr(), nb.SF_SWIZZLED, torch.cuda.current_stream().cuda_stream)
                assert stt == 0
            ms = time_call(dual, reps, graph=small)
            gbs = n_el * 3.125 / (ms * 1e-3) / 1e9
            rec[label] = {"GB/s": gbs, "us": ms * 1e3, "bytes_per_element": 3.125,
                          "frac_of_measured_copy": gbs / peaks["hbm_gbs"], "frac_of_8TBs": gbs / 8000.0}
        ms = time_call(lambda: nb.nvfp4_tensor_amax_scale(xq, out=gq), reps, graph=small)
        rec["amax"] = {"GB/s": n_el * 2.0 / (ms * 1e-3) / 1e9, "us": ms * 1e3, "bytes_per_element": 2.0}
        if n_el == 2 ** 28:
            out.update(rec)                     # the HBM figures stay at the top level of the record
        else:
            out[f"elements_2p{n_el.bit_length() - 1}"] = rec
        del xq, codes, sfs, ct, st
        torch.cuda.empty_cache()
    return out


def long_token_axis_leg(nb, dev):
    """The FFN weight-gradient product with a 65536-token contraction (Eq. 3/6): dW = dY^T X, dY 65536 x 11008,
    X 65536 x 4096, both SR-quantized in blocks along the tokens."""
    t = synth.LONG_DW
    M, K, N = t["tokens"], t["K"], t["N"]
    dY = synth.normal((M, N), 1e-4, 2005, device=dev)
    X = synth.normal((M, K), 1.0, 2006, device=dev)
    r_dy, r_x = nb.Rounding(nb.SR, 2, 1), nb.Rounding(nb.SR, 2, 2)
    dW = torch.empty((N, K), dtype=torch.float32, device=dev)
    ws = torch.empty(nb.nvfp4_linear_workspace_bytes(M, N, K, nb.LINEAR_BWD_DW), dtype=torch.uint8, device=dev)
    flops = 2.0 * M * N * K
    ms_e2e = time_call(lambda: nb.nvfp4_linear_bwd_dw(dY, X, nb.G_AMAX, rdy=r_dy, rx=r_x, out=dW, workspace=ws), 5, warm=2)
    gdy, gx = nb.nvfp4_tensor_amax_scale(dY), nb.nvfp4_tensor_amax_scale(X)
    ac, asf = nb.nvfp4_quantize(dY, True, gdy, r_dy, nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(X, True, gx, r_x, nb.SF_SWIZZLED)
    ms_q = [time_call(lambda: nb.nvfp4_quantize(dY, True, gdy, r_dy, nb.SF_SWIZZLED, codes=ac, scales=asf), 5, warm=2),
            time_call(lambda: nb.nvfp4_quantize(X, True, gx, r_x, nb.SF_SWIZZLED, codes=bc, scales=bsf), 5, warm=2)]
    ms_gemm = time_call(lambda: nb.nvfp4_gemm(ac, asf, gdy, bc, bsf, gx, out=dW), 10, warm=2)
    return {"workload": "ffn_weight_gradient_65536_tokens", "M_tokens": M, "N": N, "K": K, "flops": flops,
            "gemm_only_TFLOPS": flops / ms_gemm / 1e9, "gemm_ms": ms_gemm,
            "end_to_end_TFLOPS": flops / ms_e2e / 1e9, "end_to_end_ms": ms_e2e,
            "end_to_end_is": "amax x2 + transposed SR quantizers x2 + GEMM, through nvfp4_linear_bwd_dw",
            "transposed_sr_quantizer_GBs": {"dY": M * N * 2.5625 / ms_q[0] / 1e6, "X": M * K * 2.5625 / ms_q[1] / 1e6}}


def fused_producer_leg(nb, dev, cfg):
    """Quantization fused into the producing GEMM (no bf16/fp32 round trip): the up projection's product leaves
    its GEMM already quantized along its feature axis (nvfp4_linear_fwd_qout) and feeds the down projection
    (nvfp4_linear_fwd_qin) -- the position of the SwiGLU output in Section 5's model; the activation itself is not
    part of this library.  Against the unfused pair of nvfp4_linear_fwd calls: fp32 intermediate written, read
    back for its amax and read again by the next layer's quantizer.  Per-tensor scales are given in both arms."""
    M = cfg["tokens"]
    (_, K1, N1), (_, K2, N2) = [l for l in cfg["linears"] if l[0] in ("up", "down")]
    assert N1 == K2
    X, W1, _ = synth.linear_inputs(M, K1, N1, seed=4100, device=dev)
    _, W2, _ = synth.linear_inputs(M, K2, N2, seed=4101, device=dev)
    rt = nb.Rounding(nb.RTN)
    gx, g1, g2 = nb.nvfp4_tensor_amax_scale(X), nb.nvfp4_tensor_amax_scale(W1), nb.nvfp4_tensor_amax_scale(W2)
    H = torch.empty((M, N1), dtype=torch.float32, device=dev)
    Y = torch.empty((M, N2), dtype=torch.float32, device=dev)
    Yf = torch.empty((M, N2), dtype=torch.float32, device=dev)
    ws = torch.empty(max(nb.nvfp4_linear_workspace_bytes(M, N1, K1, nb.LINEAR_FWD), nb.nvfp4_linear_workspace_bytes(M, N2, K2, nb.LINEAR_FWD)),
                     dtype=torch.uint8, device=dev)
    nb.nvfp4_linear_fwd(X, W1, nb.G_GIVEN, gx=gx, gw=g1, rx=rt, rw=rt, out=H, workspace=ws)
    gh = nb.nvfp4_tensor_amax_scale(H)              # the consumer's per-tensor scale must be known beforehand (delayed scaling)
    hc = torch.empty((M, N1 // 2), dtype=torch.uint8, device=dev)
    hs = torch.empty(nb.nvfp4_sf_bytes(M, N1, nb.SF_SWIZZLED), dtype=torch.uint8, device=dev)

    def fused():
        nb.nvfp4_linear_fwd_qout(X, W1, gy=gh, ry=rt, gscale_mode=nb.G_GIVEN, gx=gx, gw=g1, rx=rt, rw=rt, sf_layout=nb.SF_SWIZZLED,
                                 codes=hc, scales=hs, workspace=ws)
        nb.nvfp4_linear_fwd_qin(hc, hs, gh, W2, nb.G_GIVEN, gw=g2, rw=rt, out=Yf, workspace=ws)

    W2f = W2.float()                                # exact: the fp32 arm reads the same weight values
    H16 = torch.empty((M, N1), dtype=torch.bfloat16, device=dev)

    def unfused():                                  # fp32 intermediate: the same numbers as the fused arm, bit for bit
        nb.nvfp4_linear_fwd(X, W1, nb.G_GIVEN, gx=gx, gw=g1, rx=rt, rw=rt, out=H, workspace=ws)
        nb.nvfp4_linear_fwd(H, W2f, nb.G_GIVEN, gx=gh, gw=g2, rx=rt, rw=rt, out=Y, workspace=ws)

    def unfused_bf16():                             # bf16 intermediate: half the bytes, one more rounding of H
        nb.nvfp4_linear_fwd(X, W1, nb.G_GIVEN, gx=gx, gw=g1, rx=rt, rw=rt, out=H16, workspace=ws)
        nb.nvfp4_linear_fwd(H16, W2, nb.G_GIVEN, gx=gh, gw=g2, rx=rt, rw=rt, out=Y, workspace=ws)

    ms_f, ms_b, ms_u = time_call(fused, 10), time_call(unfused_bf16, 10), time_call(unfused, 10)
    same = bool(torch.equal(Y, Yf))
    flops = 2.0 * M * (K1 * N1 + K2 * N2)
    return {"workload": "up projection (nvfp4_linear_fwd_qout) -> down projection (nvfp4_linear_fwd_qin), given per-tensor scales",
            "M": M, "K1": K1, "N1": N1, "N2": N2,
            "fused_ms": ms_f, "unfused_ms": ms_u, "time_saved_ms": ms_u - ms_f,
            "unfused_bf16_intermediate_ms": ms_b, "time_saved_vs_bf16_intermediate_ms": ms_b - ms_f,
            "fused_TFLOPS": flops / ms_f / 1e9, "unfused_TFLOPS": flops / ms_u / 1e9,
            "results_bit_identical_to_fp32_intermediate": same,
            "bytes_not_moved": M * N1 * 8,         # the fp32 intermediate is neither written nor read back
            "bytes_note": "the M x N1 fp32 intermediate: 4 B/element written by the first GEMM + 4 B/element read by the next layer's quantizer"}


def qaf_backward_leg(nb, dev, cfg):
    """The paper's fine-tuning phase (Section 5): forward in NVFP4, backward and update products in BF16.  The two BF16
    products of the first layer, W, X and dY read as they are stored (MN-major operands, no transposed copies)."""
    M = cfg["tokens"]
    name, K, N = cfg["linears"][0]
    X, W, dY = synth.linear_inputs(M, K, N, seed=4200, device=dev)
    dX = torch.empty((M, K), dtype=torch.float32, device=dev)
    dW = torch.empty((N, K), dtype=torch.float32, device=dev)
    L = nb.lib()

    def run():
        st = L.nvfp4_linear_bwd_bf16(dY.data_ptr(), W.data_ptr(), X.data_ptr(), M, N, K, dX.data_ptr(), nb.FP32,
                                     dW.data_ptr(), nb.FP32, None, 0, torch.cuda.current_stream().cuda_stream)
        assert st == 0
    ms = time_call(run, 10)
    flops = 4.0 * M * N * K
    return {"workload": f"layer '{name}' backward + update in bf16 (nvfp4_linear_bwd_bf16)", "M": M, "K": K, "N": N,
            "ms": ms, "TFLOPS": flops / ms / 1e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b", choices=["llama7b", "llama350m"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-quantizer", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the legs for the other workload configurations")
    ap.add_argument("--no-graph", action="store_true", help="launch every step kernel by kernel instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    from paper_2505_19115_b200 import binding as nb
    from paper_2505_19115_b200 import microbench

    rank, world, local = replicas.env_rank_world()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    nb.lib()                                      # fails loudly when the CUDA library is missing

    cfg = synth.LLAMA_7B if args.workload == "llama7b" else synth.LLAMA_350M
    peaks, peak_kind = load_peaks()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- the headline: resident inputs, every rank its own block (replicas; no data-path collective) ----
    block = Block(nb, cfg, dev, rank)
    M = block.M
    layers = block.layers
    sampler = ClockSampler(local).start() if rank == 0 else None
    for _ in range(args.warmup):
        block.step()
    barrier()
    # One step = 45 launches of 20-400 us: captured once into a CUDA graph (after the warm-up, so that every
    # one-time set-up inside the library is done) and replayed, which removes the launch gaps between them.
    ms, launch_mode = timed_graph(block.step, args.steps, barrier, not args.no_graph, sampler)
    clocks = sampler.stop() if rank == 0 else None
    ms = replicas.max_over_ranks(ms, dist, dev)
    err_word = nb.nvfp4_device_error_word()
    if err_word:
        raise RuntimeError(f"device error word {err_word:#x}: a kernel gave up on a bounded wait")
    flops_per_step = block.flops
    value = replicas.aggregate_throughput(flops_per_step * args.steps, world, ms * 1e-3) / 1e12
    launches_per_step = block.launches_per_step()

    # ---- roofline of the dominant kernel (the GEMM): same workload, decomposed into the C-ABI's
    #      quantize and gemm calls so that CUDA events bracket every GEMM launch; clocks sampled meanwhile ----
    rt, sr = block.rt, block.sr
    roof_sampler = ClockSampler(local, interval_s=0.002).start() if rank == 0 else None   # a short pass: sample it densely
    gemm_events, gemm_flops, gemm_bytes = [], 0.0, 0.0
    roof_steps = min(args.steps, 3)
    for it in range(roof_steps + 1):
        if it == 1 and roof_sampler is not None:
            torch.cuda.synchronize()
            roof_sampler.mark()                  # the first pass is warm-up
        for l in layers:
            for a, b, ta, tb, ra, rb, out in ((l["X"], l["W"], False, False, rt, rt, l["Y"]),
                                               (l["dY"], l["W"], False, True, sr[0], rt, l["dX"]),
                                               (l["dY"], l["X"], True, True, sr[1], sr[2], l["dW"])):
                ga, gb = nb.nvfp4_tensor_amax_scale(a), nb.nvfp4_tensor_amax_scale(b)
                ac, asf = nb.nvfp4_quantize(a, ta, ga, ra, nb.SF_SWIZZLED)
                bc, bsf = nb.nvfp4_quantize(b, tb, gb, rb, nb.SF_SWIZZLED)
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record()
                nb.nvfp4_gemm(ac, asf, ga, bc, bsf, gb, out=out)
                s1.record()
                if it > 0:
                    gemm_events.append((s0, s1))
                    gemm_flops += 2.0 * out.shape[0] * out.shape[1] * ac.shape[1] * 2
                    gemm_bytes += (ac.numel() + bc.numel()) * 1.125 + out.numel() * out.element_size()
                del ac, asf, bc, bsf
    torch.cuda.synchronize()
    roof_clocks = roof_sampler.stop() if rank == 0 else None
    gemm_ms = sum(a.elapsed_time(b) for a, b in gemm_events)
    n_gemm = len(gemm_events)
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12
    # The denominator follows from the run: each GEMM launch is timed alone, which is the burst regime while the
    # clock sampled during this pass stays within 10 % of its maximum; a run that the power cap has pulled below
    # that is measured against the sustained figure.
    roof_mhz = (roof_clocks or {}).get("sm_mhz")
    roof_max = (roof_clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz")
    burst = not (roof_mhz and roof_max) or roof_mhz >= 0.9 * roof_max
    bf16_peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    fp4_peak = bf16_peak * FP4_OVER_BF16
    fp4_sustained = peaks["bf16_tflops_sustained"] * FP4_OVER_BF16
    # the tensor pipe's own ceiling, measured now: the GEMM's instruction issued back to back on resident operands
    mma = microbench.mma_peak(stages=1024, iters=3, warmup=1) if rank == 0 else None
    issue_peak_at_clock = sms * MMA_FLOP_PER_CLK_PER_SM * roof_mhz * 1e6 / 1e12 if roof_mhz else None
    roofline = {
        "bound": "tensor", "kernel": "gemm2_nvfp4_kernel<256>", "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
        "frac": gemm_tflops / fp4_peak, "traffic": GEMM_TRAFFIC_RATIO * gemm_bytes / n_gemm,
        "traffic_basis": "ncu capture of an 8192x8192x4096 launch (0.96 of its algorithmic bytes), scaled by the "
                         "algorithmic bytes per launch of this workload",
        "algorithmic_bytes_per_launch_avg": gemm_bytes / n_gemm,
        "peak_basis": f"{peak_kind} {'burst' if burst else 'sustained'} bf16 {bf16_peak} TFLOP/s x {FP4_OVER_BF16:g} (nominal dense "
                      f"NVFP4/bf16 ratio): every GEMM launch is timed alone and the SM clock sampled during this pass had a "
                      f"median of {roof_mhz} MHz of {roof_max} ({'within' if burst else 'more than'} 10 % of the maximum)",
        "launches": n_gemm, "avg_launch_ms": gemm_ms / n_gemm, "flops_per_launch_avg": gemm_flops / n_gemm,
        "frac_of_burst_x4": gemm_tflops / (peaks["bf16_tflops"] * FP4_OVER_BF16),
        "frac_of_sustained_x4": gemm_tflops / fp4_sustained,
        "frac_of_nominal_9pf": gemm_tflops / NOMINAL_FP4_TFLOPS,
        "issue_peak_at_sampled_clock": issue_peak_at_clock,
        "frac_of_issue_peak": gemm_tflops / issue_peak_at_clock if issue_peak_at_clock else None,
        "issue_peak_basis": f"{sms} SMs x {MMA_FLOP_PER_CLK_PER_SM:g} FLOP/clk x the sampled median clock",
        "mma_peak_measured": mma,
        "frac_of_mma_peak_measured": gemm_tflops / mma["TFLOP/s"] if mma else None,
        "mma_peak_note": "tcgen05.mma kind::mxf4nvf4 (256x256x64, CTA pair) issued back to back on resident operands in this "
                         "run: the rate the tensor pipe delivers at the clock it holds under that load (implied_sm_mhz)",
        "clocks": roof_clocks,
    }

    # ---- quantizer bandwidths ----
    quant = None
    if not args.no_quantizer and rank == 0:
        for l in layers:
            l["Y"] = l["dX"] = l["dW"] = None
        torch.cuda.empty_cache()
        quant = quantizer_sweep(nb, dev, peaks, peak_kind)
    for l in layers:
        for k in ("Y", "dX", "dW"):
            if l[k] is None:
                shape = {"Y": (M, l["N"]), "dX": (M, l["K"]), "dW": (l["N"], l["K"])}[k]
                l[k] = torch.empty(shape, dtype=torch.float32, device=dev)

    # ---- the other workload configurations and modes (single GPU, rank 0; a few seconds in total) ----
    configs = None
    if not args.no_configs and rank == 0 and world == 1:
        configs = {}
        n_extra = 10
        # delayed per-tensor scales: the same step with g supplied (no amax sweep inside the timed region)
        block.compute_given_scales()
        for _ in range(2):
            block.step(nb.G_GIVEN)
        ms_g, _ = timed_graph(lambda: block.step(nb.G_GIVEN), n_extra, barrier, not args.no_graph)
        configs["step_with_given_scales"] = {
            "workload": "the headline block step with NVFP4_G_GIVEN: per-tensor scales carried over (delayed scaling), no amax pass",
            "ms_per_step": ms_g / n_extra, "TFLOPS": flops_per_step * n_extra / ms_g / 1e9,
            "gpu_launches_per_step": block.launches_per_step(nb.G_GIVEN)}
        # bf16 activations out (Y, dX), fp32 weight gradient
        del block.layers[:]
        del block, layers
        torch.cuda.empty_cache()
        blk16 = Block(nb, cfg, dev, rank, act_dtype=torch.bfloat16)
        for _ in range(2):
            blk16.step()
        ms_b, _ = timed_graph(blk16.step, n_extra, barrier, not args.no_graph)
        configs["step_with_bf16_activations"] = {
            "workload": "the headline block step with bf16 Y and dX and fp32 dW (amax inside the calls)",
            "ms_per_step": ms_b / n_extra, "TFLOPS": flops_per_step * n_extra / ms_b / 1e9}
        del blk16.layers[:]
        del blk16
        torch.cuda.empty_cache()
        # the 350M-class block (or the 7B one when that is not the headline)
        other = synth.LLAMA_350M if args.workload == "llama7b" else synth.LLAMA_7B
        blk_o = Block(nb, other, dev, rank)
        for _ in range(3):
            blk_o.step()
        n_o = 20
        ms_o, _ = timed_graph(blk_o.step, n_o, barrier, not args.no_graph)
        configs["other_block"] = {
            "workload": ("llama350m" if args.workload == "llama7b" else "llama7b") + "_block_linears_fwd_bwd",
            "tokens": other["tokens"], "hidden": other["hidden"], "ms_per_step": ms_o / n_o,
            "TFLOPS": blk_o.flops * n_o / ms_o / 1e9, "flops_per_step": blk_o.flops}
        del blk_o.layers[:]
        del blk_o
        torch.cuda.empty_cache()
        configs["long_token_axis_weight_gradient"] = long_token_axis_leg(nb, dev)
        torch.cuda.empty_cache()
        configs["quantization_fused_into_producer"] = fused_producer_leg(nb, dev, synth.LLAMA_7B)
        torch.cuda.empty_cache()
        configs["qaf_backward_bf16"] = qaf_backward_leg(nb, dev, synth.LLAMA_7B)
        torch.cuda.empty_cache()
        err_word = nb.nvfp4_device_error_word()
        if err_word:
            raise RuntimeError(f"device error word {err_word:#x} in the configuration legs")
        block = Block(nb, cfg, dev, rank)          # back to the headline block for the end-to-end leg
        layers = block.layers

    # ---- end to end through the C ABI with host buffers (H2D of every input, D2H of every output) ----
    e2e = None
    if not args.no_e2e:
        host_in = [{k: l[k].cpu().pin_memory() for k in ("X", "W", "dY")} for l in layers]
        max_out = {k: max(l[k].numel() for l in layers) for k in ("Y", "dX", "dW")}
        host_out = {k: torch.empty(n, dtype=torch.float32).pin_memory() for k, n in max_out.items()}
        h2d = sum(t.numel() * t.element_size() for h in host_in for t in h.values())
        d2h = sum(l[k].numel() * 4 for l in layers for k in ("Y", "dX", "dW"))

        # Three streams: inputs arrive on one, the layer calls run on the second, results leave on the third,
        # so that the PCIe transfers (full duplex) overlap each other and the compute.  Events keep the order:
        # a layer computes after its inputs landed and after its previous outputs were read back; an input
        # buffer is overwritten only after the layer that read it has run.
        s_in, s_cmp, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in layers]
        ev_done = [torch.cuda.Event() for _ in layers]
        ev_out = [torch.cuda.Event() for _ in layers]
        first = [True]

        def e2e_step():
            for i, (l, h) in enumerate(zip(layers, host_in)):
                with torch.cuda.stream(s_in):
                    if not first[0]:
                        s_in.wait_event(ev_done[i])
                    for k in ("X", "W", "dY"):
                        l[k].copy_(h[k], non_blocking=True)
                    ev_in[i].record(s_in)
                with torch.cuda.stream(s_cmp):
                    s_cmp.wait_event(ev_in[i])
                    if not first[0]:
                        s_cmp.wait_event(ev_out[i])
                    block.layer(l, nb.G_AMAX)
                    ev_done[i].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[i])
                    for k in ("Y", "dX", "dW"):
                        host_out[k][:l[k].numel()].copy_(l[k].view(-1), non_blocking=True)
                    ev_out[i].record(s_out)
            first[0] = False

        def e2e_join():
            cur = torch.cuda.current_stream()
            for st_ in (s_in, s_cmp, s_out):
                cur.wait_stream(st_)

        e2e_steps = max(1, min(args.steps, 3))
        for st_ in (s_in, s_cmp, s_out):
            st_.wait_stream(torch.cuda.current_stream())
        e2e_step()
        e2e_join()
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for st_ in (s_in, s_cmp, s_out):
            st_.wait_stream(torch.cuda.current_stream())
        for _ in range(e2e_steps):
            e2e_step()
        e2e_join()
        f1.record()
        barrier()
        ems = f0.elapsed_time(f1)
        ems = replicas.max_over_ranks(ems, dist, dev)
        e2e = {"value": flops_per_step * e2e_steps * world / (ems * 1e-3) / 1e12, "unit": "TFLOPS",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "ms_per_step": ems / e2e_steps}
        del host_in, host_out

    # ---- the oracle on the host cores, bounded samples, after every timed GPU region ----
    cpu = None
    if rank == 0 and not args.no_cpu and world == 1:
        cpu = cpu_baseline_record(cfg)

    if rank == 0:
        ms_step = ms / args.steps
        mhz = (clocks or {}).get("sm_mhz")
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step,
            "ms_x_mhz_per_step": ms_step * mhz if mhz else None,      # separates the power-capped regime from the burst one
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "nvfp4 (e2m1 x ue4m3 block scales), fp32 accumulate and output",
            "data": "synthetic",
            "config": {"workload": "llama7b_block_linears_fwd_bwd" if args.workload == "llama7b" else "llama350m_block_linears_fwd_bwd",
                       "tokens": M, "hidden": cfg["hidden"], "linears": [[n, k, o] for n, k, o in cfg["linears"]],
                       "products_per_step": 15, "rounding": "RtN forward, Philox SR backward/update",
                       "per_tensor_scale": "amax/(6*448), computed once per tensor inside the calls",
                       "launch": launch_mode,
                       "fusion": "nvfp4_linear_fwd_save + nvfp4_linear_bwd_saved: X, W, dY each read once per pass, both orientations quantized from that read",
                       "l2": f"inputs exceed L2: {sum(2 * M * (k + o) + 2 * k * o for _, k, o in cfg['linears']) / 2 ** 20:.0f} MiB of operands per step, fp32 outputs on top",
                       "timed_region_s": ms * 1e-3,
                       "parallelism": "replicas only (one GPU per rank, no data-path collective)"},
            "pct_of_fp4_peak": {"of_nominal_9pf": value / world / NOMINAL_FP4_TFLOPS * 100,
                                f"of_{peak_kind}_sustained_x4": value / world / fp4_sustained * 100,
                                f"of_{peak_kind}_burst_x4": value / world / (peaks["bf16_tflops"] * FP4_OVER_BF16) * 100},
            "roofline": roofline, "quantizer": quant, "configs": configs, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
