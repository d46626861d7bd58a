#!/usr/bin/env python
"""Benchmark of the NVFP4 quantize-then-GEMM hot path on B200.

One "step" is one pass of the whole hot path over one Llama-7B-shaped transformer block's five
linear layers (tokens 16384, hidden 4096): for each layer the forward product (Eq. 1/4), the
input-gradient product (Eq. 2/5) and the weight-gradient product (Eq. 3/6), each with its
per-tensor amax passes, its two operand quantizations and its block-scaled GEMM, all through
the C-ABI entry points nvfp4_linear_fwd / nvfp4_linear_bwd_dx / nvfp4_linear_bwd_dw.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample of
the same workload instead.
"""
import argparse
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
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic of the GEMM kernel from the committed ncu capture (profiles/gemm2_nvfp4_kernel_8192x8192x4096.md):
# 83.0 MB read + 212.2 MB written for 306.2 MB of algorithmic bytes (operand codes and scales + fp32 output).
# GEMM traffic follows bytes, not FLOPs, so the workload's figure is this ratio times its own algorithmic bytes.
GEMM_TRAFFIC_RATIO = (83.05 + 212.17) / 306.2


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
    thread (every 10 ms) while the timed region runs."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, device_index):
        self.idx = device_index
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
                time.sleep(0.01)
        except Exception as e:  # the number is still reported, without a clock record
            self.error = repr(e)

    def start(self):
        import threading
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

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
# reference arm: the CPU oracle on a bounded sample
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(cfg, rows=256, seed=2004):
    """One bounded sample of the workload on the host: the first layer's forward product for the
    first `rows` tokens (quantize those rows of X, quantize all of W, dequantize-then-matmul)."""
    from oracle import binding as ob
    name, K, N = cfg["linears"][0]
    X = synth.normal((rows, K), 1.0, seed, device="cpu").float().numpy()
    W = synth.normal((N, K), 0.02, seed + 1, device="cpu").float().numpy()
    t0 = time.perf_counter()
    gx, gw = ob.tensor_amax_scale(X), ob.tensor_amax_scale(W)
    xc, xs = ob.quantize(X, g=gx)
    wc, ws = ob.quantize(W, g=gw)
    ob.gemm(xc, xs, gx, wc, ws, gw, want_T=False)
    dt = time.perf_counter() - t0
    flops = 2.0 * rows * K * N
    return flops, dt, f"layer '{name}' forward product on the first {rows} of {cfg['tokens']} tokens " \
                      f"(quantize X rows + all of W, dequantize-then-matmul in double)"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import binding as ob
    cfg = synth.LLAMA_7B
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample_step(cfg)
    flops = secs = 0.0
    sample = ""
    for _ in range(args.steps):
        f, dt, sample = oracle_sample_step(cfg)
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
    ap.add_argument("--no-graph", action="store_true", help="launch every step kernel by kernel instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    from paper_2505_19115_b200 import binding as nb

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
    M = cfg["tokens"]
    peaks, peak_kind = load_peaks()

    # ---- resident inputs: every rank has its own block (replicas; no data-path collective) ----
    layers = []
    for li, (name, K, N) in enumerate(cfg["linears"]):
        X, W, dY = synth.linear_inputs(M, K, N, seed=replicas.replica_seed(4000 + 10 * li, rank), device=dev)
        layers.append(dict(name=name, K=K, N=N, X=X, W=W, dY=dY,
                           Y=torch.empty((M, N), dtype=torch.float32, device=dev),
                           dX=torch.empty((M, K), dtype=torch.float32, device=dev),
                           dW=torch.empty((N, K), dtype=torch.float32, device=dev)))
    ws_bytes = max(nb.nvfp4_linear_fused_workspace_bytes(M, l["N"], l["K"], w) for l in layers
                   for w in (nb.FUSED_FWD_SAVE, nb.FUSED_BWD_SAVED))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    saved = torch.empty(max(nb.nvfp4_linear_saved_bytes(M, l["N"], l["K"]) for l in layers), dtype=torch.uint8, device=dev)
    rt = nb.Rounding(nb.RTN)
    sr = [nb.Rounding(nb.SR, 0, o) for o in range(3)]      # distinct offsets per SR site
    in_bytes = sum(t.numel() * t.element_size() for l in layers for t in (l["X"], l["W"], l["dY"]))

    def layer_fwd_bwd(l):
        # forward (Eq. 1/4) keeping Q(X^T), Q(W^T); backward + update (Eq. 2/5, 3/6) from one read of dY.
        # Each tensor's amax is taken once, each tensor is read once per pass.
        nb.nvfp4_linear_fwd_save(l["X"], l["W"], nb.G_AMAX, rx=rt, rw=rt, rxt=sr[2], rwt=rt, out=l["Y"], saved=saved,
                                 workspace=ws)
        nb.nvfp4_linear_bwd_saved(l["dY"], saved, l["K"], nb.G_AMAX, rdy=sr[0], rdyt=sr[1], dX=l["dX"], dW=l["dW"],
                                  workspace=ws)

    def step():
        for l in layers:
            layer_fwd_bwd(l)

    launches_per_step = len(layers) * (3 + 3 + 3)         # 3 amax sweeps, 3 dual quantizers, 3 GEMMs per layer
    flops_per_step = block_flops(cfg)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    # One step = 60 launches of 20-400 us: captured once into a CUDA graph (after the warm-up, so that every
    # one-time set-up inside the library is done) and replayed, which removes the launch gaps between them.
    # The graph holds exactly the calls of step(), on the same buffers.
    run_step, launch_mode = step, "stream"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()                      # one more untimed step, through the graph
            run_step, launch_mode = graph.replay, "cuda_graph"
        except Exception as e:                  # capture refused: time the plain launches and say so
            launch_mode = f"stream (graph capture failed: {type(e).__name__})"
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark()
    e0.record()
    for _ in range(args.steps):
        run_step()
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    ms = replicas.max_over_ranks(ms, dist, dev)
    err_word = nb.nvfp4_device_error_word()
    if err_word:
        raise RuntimeError(f"device error word {err_word:#x}: a kernel gave up on a bounded wait")
    value = replicas.aggregate_throughput(flops_per_step * args.steps, world, ms * 1e-3) / 1e12

    # ---- roofline of the dominant kernel (the GEMM): same workload, decomposed into the C-ABI's
    #      quantize and gemm calls so that CUDA events bracket every GEMM launch ----
    def decomposed_ops(l):
        ops = []
        for kind, a, b, ta, tb, ra, rb, out in (("fwd", l["X"], l["W"], False, False, rt, rt, l["Y"]),
                                                 ("dx", l["dY"], l["W"], False, True, sr[0], rt, l["dX"]),
                                                 ("dw", l["dY"], l["X"], True, True, sr[1], sr[2], l["dW"])):
            ops.append((a, b, ta, tb, ra, rb, out))
        return ops

    gemm_events = []
    gemm_flops = 0.0
    gemm_bytes = 0.0
    roof_steps = min(args.steps, 3)
    for it in range(roof_steps + 1):
        for l in layers:
            for a, b, ta, tb, ra, rb, out in decomposed_ops(l):
                ga, gb = nb.nvfp4_tensor_amax_scale(a), nb.nvfp4_tensor_amax_scale(b)
                ac, asf = nb.nvfp4_quantize(a, ta, ga, ra, nb.SF_SWIZZLED)
                bc, bsf = nb.nvfp4_quantize(b, tb, gb, rb, nb.SF_SWIZZLED)
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record()
                nb.nvfp4_gemm(ac, asf, ga, bc, bsf, gb, out=out)
                s1.record()
                if it > 0:                       # first pass is warm-up
                    gemm_events.append((s0, s1))
                    gemm_flops += 2.0 * out.shape[0] * out.shape[1] * ac.shape[1] * 2
                    gemm_bytes += (ac.numel() + bc.numel()) * 1.125 + out.numel() * out.element_size()
                del ac, asf, bc, bsf
    torch.cuda.synchronize()
    gemm_ms = sum(a.elapsed_time(b) for a, b in gemm_events)
    n_gemm = len(gemm_events)
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12
    fp4_peak = peaks["bf16_tflops_sustained"] * FP4_OVER_BF16
    roofline = {
        "bound": "tensor", "kernel": "gemm2_nvfp4_kernel<256>", "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
        "frac": gemm_tflops / fp4_peak, "traffic": GEMM_TRAFFIC_RATIO * gemm_bytes / n_gemm,
        "traffic_basis": "ncu capture of an 8192x8192x4096 launch (0.96 of its algorithmic bytes), scaled by the "
                         "algorithmic bytes per launch of this workload",
        "algorithmic_bytes_per_launch_avg": gemm_bytes / n_gemm,
        "peak_basis": f"{peak_kind} sustained bf16 {peaks['bf16_tflops_sustained']} TFLOP/s x {FP4_OVER_BF16:g} "
                      f"(nominal dense NVFP4/bf16 ratio); burst basis {peaks['bf16_tflops'] * FP4_OVER_BF16:.0f}; nominal 9000",
        "launches": n_gemm, "avg_launch_ms": gemm_ms / n_gemm, "flops_per_launch_avg": gemm_flops / n_gemm,
        "frac_of_nominal_9pf": gemm_tflops / 9000.0,
    }

    # ---- quantizer bandwidth at 2^28 elements (heavy-tailed inputs), bytes = 2 + 0.5 + 1/16 per element ----
    quant = None
    if not args.no_quantizer and rank == 0:
        for l in layers:
            l["Y"] = l["dX"] = l["dW"] = None
        torch.cuda.empty_cache()
        n_el = 2 ** 28
        xq = synth.heavy_tailed(synth.square_shape(n_el), seed=1002, device=dev)
        gq = nb.nvfp4_tensor_amax_scale(xq)
        codes = torch.empty((xq.shape[0], xq.shape[1] // 2), dtype=torch.uint8, device=dev)
        sfs = torch.empty(nb.nvfp4_sf_bytes(xq.shape[0], xq.shape[1], nb.SF_SWIZZLED), dtype=torch.uint8, device=dev)
        quant = {"elements": n_el, "bytes_per_element": 2.5625, "peak_hbm_gbs": peaks["hbm_gbs"], "peak_kind": peak_kind}
        for label, tr, rr in (("row_rtn", False, rt), ("row_sr", False, nb.Rounding(nb.SR, 1, 0)),
                              ("transposed_rtn", True, rt), ("transposed_sr", True, nb.Rounding(nb.SR, 1, 0))):
            for _ in range(3):
                nb.nvfp4_quantize(xq, tr, gq, rr, nb.SF_SWIZZLED, codes=codes, scales=sfs)
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 10
            q0.record()
            for _ in range(reps):
                nb.nvfp4_quantize(xq, tr, gq, rr, nb.SF_SWIZZLED, codes=codes, scales=sfs)
            q1.record()
            torch.cuda.synchronize()
            gbs = n_el * 2.5625 * reps / (q0.elapsed_time(q1) * 1e-3) / 1e9
            quant[label] = {"GB/s": gbs, "frac_of_measured_copy": gbs / peaks["hbm_gbs"], "frac_of_8TBs": gbs / 8000.0}
        # both orientations from one read (the fused layer's quantizer): 2 + 2 * 0.5625 bytes per element
        L = nb.lib()
        import ctypes as C
        ct = torch.empty((xq.shape[1], xq.shape[0] // 2), dtype=torch.uint8, device=dev)
        st = torch.empty(nb.nvfp4_sf_bytes(xq.shape[1], xq.shape[0], nb.SF_SWIZZLED), dtype=torch.uint8, device=dev)
        for label, r1, r2 in (("dual_rtn", rt, rt), ("dual_sr", nb.Rounding(nb.SR, 1, 0), nb.Rounding(nb.SR, 1, 1))):
            def dual():
                stt = L.nvfp4_quantize_dual(xq.data_ptr(), nb.BF16, xq.shape[0], xq.shape[1], xq.stride(0), gq.data_ptr(),
                                            C.byref(r1), codes.data_ptr(), sfs.data_ptr(), C.byref(r2), ct.data_ptr(),
                                            st.data_ptr(), nb.SF_SWIZZLED, torch.cuda.current_stream().cuda_stream)
                assert stt == 0
            for _ in range(3):
                dual()
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
            for _ in range(10):
                dual()
            q1.record()
            torch.cuda.synchronize()
            gbs = n_el * 3.125 * 10 / (q0.elapsed_time(q1) * 1e-3) / 1e9
            quant[label] = {"GB/s": gbs, "bytes_per_element": 3.125, "frac_of_measured_copy": gbs / peaks["hbm_gbs"],
                            "frac_of_8TBs": gbs / 8000.0}
        del xq, codes, sfs, ct, st
        torch.cuda.empty_cache()

    # ---- end to end through the C ABI with host buffers (H2D of every input, D2H of every output) ----
    e2e = None
    if not args.no_e2e:
        for l in layers:
            for k in ("Y", "dX", "dW"):
                if l[k] is None:
                    shape = {"Y": (M, l["N"]), "dX": (M, l["K"]), "dW": (l["N"], l["K"])}[k]
                    l[k] = torch.empty(shape, dtype=torch.float32, device=dev)
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
                    layer_fwd_bwd(l)
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

    # ---- the oracle on the host cores, bounded sample ----
    cpu = None
    if rank == 0 and not args.no_cpu and world == 1:
        from oracle import binding as ob
        f = secs = 0.0
        sample = ""
        for _ in range(2):
            ff, dt, sample = oracle_sample_step(cfg)
            f += ff
            secs += dt
        cpu = {"value": f / secs / 1e12, "unit": "TFLOPS", "cores": ob.host_threads(), "kind": "oracle",
               "sample": sample + f"; 2 repetitions, {secs:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "nvfp4 (e2m1 x ue4m3 block scales), fp32 accumulate and output",
            "data": "synthetic",
            "config": {"workload": "llama7b_block_linears_fwd_bwd" if args.workload == "llama7b" else "llama350m_block_linears_fwd_bwd",
                       "tokens": M, "hidden": cfg["hidden"], "linears": [[n, k, o] for n, k, o in cfg["linears"]],
                       "products_per_step": 15, "rounding": "RtN forward, Philox SR backward/update",
                       "per_tensor_scale": "amax/(6*448), computed once per tensor inside the calls",
                       "launch": launch_mode,
                       "fusion": "nvfp4_linear_fwd_save + nvfp4_linear_bwd_saved: X, W, dY each read once per pass, both orientations quantized from that read",
                       "l2": f"inputs exceed L2: {in_bytes / 2 ** 20:.0f} MiB of operands per step, fp32 outputs on top",
                       "parallelism": "replicas only (one GPU per rank, no data-path collective)"},
            "pct_of_fp4_peak": {"of_nominal_9pf": value / world / 9000.0 * 100,
                                f"of_{peak_kind}_sustained_x4": value / world / fp4_peak * 100},
            "roofline": roofline, "quantizer": quant, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
