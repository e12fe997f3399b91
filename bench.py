#!/usr/bin/env python
"""Benchmark of the MX+ hot path on B200: activation quantize (bf16 -> MXFP4+) followed by
the block-scaled GEMM against pre-quantized MXFP4+ weights.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg5|cfg4|small] [--no-targets] [--parts] [--only PART]

One "step" = mxp_quantize(A) + mxp_gemm(A_q, W_q) on one batch of synthetic activations.
Prints ONE JSON line (rank 0).  Besides the timed steps the line carries `sustained` (the same
step after at least 300 ms of dense load, whatever --steps was) and, as its last key,
`targets`: the quantize, decode and prefill figures of every configuration against their
rooflines, MXFP4+ beside plain MXFP4.  `--parts` adds the long per-kernel list.
`--impl reference` times the CPU oracle instead, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (M, N, K, label)
    "cfg5": (8192, 28672, 8192, "prefill 8192x8192x28672 (Llama-70B MLP-like), both operands MX+, quantize->GEMM"),
    "cfg4": (2048, 4096, 4096, "prefill 2048x4096x4096, both operands MX+, quantize->GEMM"),
    "small": (256, 512, 512, "small smoke shape, both operands MX+, quantize->GEMM"),
}
METRIC = "MX+ quantize->GEMM throughput (prefill, both operands MXFP4+, 2*M*N*K per step)"
UNIT = "TFLOP/s"
NOMINAL_FP4_OVER_BF16 = 4.0  # 9 PF dense FP4 vs 2.25 PF dense bf16
NOMINAL_FP8_OVER_BF16 = 2.0  # 4.5 PF dense for 8-bit containers (kind::mxf8f6f4)
# dram__bytes_read.sum + dram__bytes_write.sum of one gemm_tc_stream_kernel<wide> launch, from
# single-pass ncu captures of this program (summaries under profiles/); bytes per launch.
NCU_DRAM_TRAFFIC = {"cfg5": 531.75e6 + 441.83e6, "cfg4": 19.82e6 + 64.8e3}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "src": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "src": "fallback"}


# ------------------------------------------------------------------------- clocks sampling
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self, upto=None):
        """Ends the sampling; the summary covers the first `upto` samples (default: all)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        return self.summary(self.lines if upto is None else self.lines[:max(upto, 1)])

    @staticmethod
    def summary(lines):
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_run(M, N, K, rows_a=32, rows_b=2048, seed=4):
    """One oracle pass on a bounded sample of the workload: quantize rows_a activation rows
    and rows_b weight rows to MXFP4+, decode them, multiply in fp64.  Returns (seconds, flops)."""
    import oracle
    from paper_2510_14557_b200 import synth
    rows_a, rows_b = min(rows_a, M), min(rows_b, N)
    a_bits = synth.f32_to_bf16_bits(synth.activations_normal(rows_a, K, seed, 0.01, 30.0))
    w_bits = synth.f32_to_bf16_bits(synth.weights(rows_b, K, seed + 100))
    t0 = time.perf_counter()
    qa = oracle.quantize(a_bits, oracle.MODE_MXFP4_PLUS, bf16_bits=True)
    qw = oracle.quantize(w_bits, oracle.MODE_MXFP4_PLUS, bf16_bits=True)
    da = oracle.dequantize(*qa, oracle.MODE_MXFP4_PLUS)
    dw = oracle.dequantize(*qw, oracle.MODE_MXFP4_PLUS)
    oracle.gemm_fp64(da, dw)
    dt = time.perf_counter() - t0
    return dt, 2.0 * rows_a * rows_b * K


def cpu_baseline(M, N, K):
    import oracle
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    rows_a, rows_b = 32, 2048
    dt, fl = oracle_sample_run(M, N, K, rows_a, rows_b)
    # grow the sample (more activation rows) until it is about 10 s of CPU work
    for _ in range(3):
        if dt >= 8.0 or rows_a >= M:
            break
        rows_a = min(M, max(rows_a + 1, int(rows_a * min(16.0, 12.0 / max(dt, 0.05)))))
        dt, fl = oracle_sample_run(M, N, K, rows_a, rows_b)
    out = {"value": fl / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": "%d activation rows x %d weight rows x K=%d of the workload "
                     "(quantize both to MXFP4+, decode, fp64 GEMM), %.1f s, %d OpenMP threads"
                     % (min(rows_a, M), min(rows_b, N), K, dt, cores)}
    # the same on one thread, on a sample cut down by the thread count
    oracle.set_threads(1)
    rows_1 = max(1, min(rows_a, M) // max(1, cores))
    dt1, fl1 = oracle_sample_run(M, N, K, rows_1, rows_b)
    oracle.set_threads(cores)
    out["single_thread"] = {"value": fl1 / dt1 / 1e12, "unit": UNIT, "cores": 1,
                            "sample": "%d activation rows x %d weight rows x K=%d, %.1f s"
                                      % (rows_1, min(rows_b, N), K, dt1)}
    return out


def run_reference(args, M, N, K, label):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    rows_a, rows_b = 16, 1024
    times = []
    for i in range(args.warmup + args.steps):
        dt, fl = oracle_sample_run(M, N, K, rows_a, rows_b)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = fl / (ms / 1e3) / 1e12
    sample = "%d activation rows x %d weight rows x K=%d per step" % (min(rows_a, M), min(rows_b, N), K)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": label, "M": M, "N": N, "K": K, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------- multi-rank glue
def aggregate(ms_local: float, flops_local: float, dist=None):
    """Max time over ranks and summed work (weak scaling: every rank runs its own batch)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_local, flops_local
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    f = torch.tensor([flops_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f.item())


# ------------------------------------------------------------------------- GPU legs
def dev_bf16(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def time_loop(fn, iters, warmup=3):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters  # ms


def parts(mxp, synth, peaks, only=None, iters_scale=1.0):
    """Per-config numbers: quantize (config 2), decode GEMM (config 3), prefill GEMM (config 4),
    each in MXFP4+ and in plain MXFP4.  `only` restricts the run to one of
    "quantize" / "decode" / "prefill" (used for profiler captures of a single kernel)."""
    import torch
    out = {}
    if only in (None, "quantize"):
        out.update(part_quantize(mxp, synth, peaks, max(2, int(20 * iters_scale))))
    if only in (None, "decode"):
        out.update(part_decode(mxp, synth, peaks, max(2, int(40 * iters_scale))))
    if only in (None, "prefill"):
        out.update(part_prefill(mxp, synth, peaks, max(1, int(10 * iters_scale))))
    if only == "prefill_cfg4":
        out.update(part_small_prefill(mxp, synth, max(1, int(4 * iters_scale))))
    if only == "decode_tc":
        out.update(part_decode_tc(mxp, synth, max(1, int(4 * iters_scale))))
    return out


def part_small_prefill(mxp, synth, iters):
    """Config 4 through mxp_gemm_prepacked for the four mode pairs, a few launches each: a
    case small enough for multi-pass profiler captures of the streamed GEMM kernel."""
    import torch
    out = {}
    a_bits, w_bits = synth.config4()
    a, w = dev_bf16(a_bits), dev_bf16(w_bits)
    M, K = a.shape
    N = w.shape[0]
    d = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(mxp.mxp_gemm_workspace_bytes(M, N, K, False, 1, 1), dtype=torch.uint8, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for name, am, bm in (("plain", 0, 0), ("A+", 1, 0), ("W+", 0, 1), ("both", 1, 1)):
        pa, pw = mxp.mxp_quantize(a, am), mxp.mxp_quantize(w, bm)
        pre = mxp.mxp_gemm_prepack(pw, mxp.mxp_gemm_prepack_form(am, bm))
        ms = timed_flushed(lambda: mxp.mxp_gemm_prepacked(pa, pw, pre, out=d, workspace=ws), iters, flush, pre=1)
        out["prefill_cfg4_" + name] = {"us": ms * 1e3}
    return out


def part_decode_tc(mxp, synth, iters):
    """Config 3 at M = 1 on the FP4 tensor-path decode kernel, eight weight copies, a few eager
    launches per mode: the case for profiler captures of that kernel."""
    import torch
    out = {}
    a16, w_bits = synth.config3(1)
    w = dev_bf16(w_bits)
    a = dev_bf16(a16)
    N, K = w.shape
    d = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(max(256, mxp.mxp_gemm_decode_workspace_bytes(1, K)), dtype=torch.uint8, device="cuda")
    for name, mode in (("mxfp4+", mxp.MODE_MXFP4_PLUS), ("mxfp4", mxp.MODE_MXFP4)):
        tiled = [mxp.mxp_gemm_decode_prepack(mxp.mxp_quantize(w, mode)) for _ in range(8)]
        st = {"i": 0}

        def run():
            mxp.mxp_gemm_decode_prepacked(a, tiled[st["i"] % 8], out=d, workspace=ws)
            st["i"] += 1
        ms = time_loop(run, 8 * iters, warmup=8)
        out["decode_tc_cfg3_M1_" + name] = {"us": ms * 1e3}
        del tiled
    return out


def part_quantize(mxp, synth, peaks, iters):
    import torch
    out = {}
    # ---- config 2: quantize 8192 x 8192 bf16 (inputs larger than L2: 134 MB read per launch)
    hbm = peaks["hbm_gbs"]
    x = dev_bf16(synth.config2())
    n = x.numel()
    for name, mode in (("mxfp4+", mxp.MODE_MXFP4_PLUS), ("mxfp4", mxp.MODE_MXFP4),
                       ("mxfp4++", mxp.MODE_MXFP4_PP), ("mxfp6+", mxp.MODE_MXFP6_PLUS),
                       ("mxfp6", mxp.MODE_MXFP6), ("mxfp8+", mxp.MODE_MXFP8_PLUS),
                       ("mxfp8", mxp.MODE_MXFP8)):
        buf = mxp.alloc_packed(x.shape[0], x.shape[1], mode, index_for_mxfp4=False)
        ms = time_loop(lambda: mxp.mxp_quantize(x, mode, out=buf), iters)
        # bf16 in; element codes, one scale byte (and one index byte) per block of 32 out
        nbytes = n * (2 + mxp.binding.element_bits(mode) / 8 + 1 / 32 + (1 / 32 if buf.bm_index is not None else 0))
        gbs = nbytes / ms / 1e6
        out["quantize_cfg2_" + name] = {"us": ms * 1e3, "GB/s": gbs, "frac_hbm": gbs / hbm}
    # ---- NVFP4 / NVFP4+ (blocks of 16, E4M3 scale): 2 B in, 4 bits + 1/16 B (+ 1/32 B) out
    for name, plus in (("nvfp4+", True), ("nvfp4", False)):
        ms = time_loop(lambda: mxp.mxp_nvfp4_quantize(x, 2.0 ** -8, plus), iters)
        nbytes = n * (2 + 0.5 + 1 / 16 + (1 / 32 if plus else 0))
        gbs = nbytes / ms / 1e6
        out["quantize_cfg2_" + name] = {"us": ms * 1e3, "GB/s": gbs, "frac_hbm": gbs / hbm}
    # ---- the same with channel reordering fused in: ordering built by the library's rule from
    # per-channel outlier counts (|x| > 3 sigma) of a 512-row sample of the input
    sample = x[:512].float()
    counts = (sample.abs() > 3.0 * sample.std()).sum(dim=0).cpu()
    order = mxp.mxp_channel_order(counts).cuda()
    for name, mode in (("mxfp4+", mxp.MODE_MXFP4_PLUS), ("mxfp4", mxp.MODE_MXFP4)):
        buf = mxp.alloc_packed(x.shape[0], x.shape[1], mode, index_for_mxfp4=False)
        ms = time_loop(lambda: mxp.mxp_quantize_reordered(x, order, mode, out=buf), iters)
        nbytes = n * (2 + 0.5 + 1 / 32 + (1 / 32 if buf.bm_index is not None else 0))
        gbs = nbytes / ms / 1e6
        out["quantize_reordered_cfg2_" + name] = {"us": ms * 1e3, "GB/s": gbs, "frac_hbm": gbs / hbm}
    return out


def part_decode(mxp, synth, peaks, iters):
    import torch
    out = {}
    hbm = peaks["hbm_gbs"]
    # ---- config 3: weight-only decode GEMM; rotate over 8 weight copies (> L2) between launches
    for name, mode in (("mxfp4+", mxp.MODE_MXFP4_PLUS), ("mxfp4", mxp.MODE_MXFP4),
                       ("mxfp4++", mxp.MODE_MXFP4_PP)):
        a16, w_bits = synth.config3(16)
        w = dev_bf16(w_bits)
        copies = []
        for _ in range(8):
            copies.append(mxp.mxp_quantize(w, mode))
        wbytes = 11008 * 4096 * (0.5 + 1 / 32 + (1 / 32 if mode != mxp.MODE_MXFP4 else 0))
        cases = [(1, None), (8, None), (16, None)] if mode != mxp.MODE_MXFP4_PP else [(1, None)]
        for M, kern in cases:
            a = dev_bf16(a16[:M].copy())
            d = torch.empty((M, 11008), dtype=torch.bfloat16, device="cuda")
            state = {"i": 0}
            key = "decode_cfg3_M%d_%s" % (M, name) + ("" if kern is None else "_kernel-" + kern)

            def run():
                mxp.mxp_gemm(a, copies[state["i"] % 8], out=d)
                state["i"] += 1
            ms = time_loop(run, iters, warmup=8)
            gbs = (wbytes + M * 4096 * 2 + M * 11008 * 2) / ms / 1e6
            out[key] = {"us": ms * 1e3, "GB/s": gbs, "frac_hbm": gbs / hbm}
            if True:
                # the same eight launches replayed from a CUDA graph: what a decode loop that
                # captures its layers sees (less launch gap between the kernels)
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    for _ in range(8):
                        run()
                torch.cuda.current_stream().wait_stream(side)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for _ in range(8):
                        run()
                ms_g = time_loop(graph.replay, max(1, iters // 8), warmup=2) / 8
                out[key]["us_cuda_graph"] = ms_g * 1e3
                out[key]["frac_hbm_cuda_graph"] = (wbytes + M * 4096 * 2 + M * 11008 * 2) / ms_g / 1e6 / hbm
            if kern is None:
                # the eight launches as a chain of programmatic dependents (each grid's weight
                # stream starts while the previous grid drains; activations and output stay
                # ordered): what a captured decode loop over constant weights can use
                def run_chained():
                    mxp.mxp_gemm_decode_chained(a, copies[state["i"] % 8], d)
                    state["i"] += 1
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    for _ in range(8):
                        run_chained()
                torch.cuda.current_stream().wait_stream(side)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for _ in range(8):
                        run_chained()
                ms_c = time_loop(graph.replay, max(1, iters // 8), warmup=2) / 8
                out[key]["us_cuda_graph_chained"] = ms_c * 1e3
                out[key]["frac_hbm_cuda_graph_chained"] = (wbytes + M * 4096 * 2 + M * 11008 * 2) / ms_c / 1e6 / hbm
        del copies, w
    # ---- weight-only form at prefill sizes (the paper's matmul table: N = K = 4096, M up to
    # 4096): bf16 activations on the block-scaled tensor-core kernel as two E4M3 planes; the
    # yardstick is the measured bf16 GEMM rate, what "convert the weights, then a bf16 GEMM" runs at
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for M in (256, 2048, 4096):
        a_bits, w_bits = synth.config3(M, 4096, 4096, seed=7)
        a, w = dev_bf16(a_bits), dev_bf16(w_bits)
        d = torch.empty((M, 4096), dtype=torch.bfloat16, device="cuda")
        for name, mode in (("mxfp4+", mxp.MODE_MXFP4_PLUS), ("mxfp4", mxp.MODE_MXFP4)):
            pw = mxp.mxp_quantize(w, mode)
            ws = torch.zeros(mxp.mxp_gemm_workspace_bytes(M, 4096, 4096, True, 0, mode),
                             dtype=torch.uint8, device="cuda")
            n_it = max(2, iters // 4)
            tot = 0.0
            for i in range(n_it + 2):
                flush.fill_(i & 255)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                mxp.mxp_gemm(a, pw, out=d, workspace=ws)
                e1.record()
                torch.cuda.synchronize()
                if i >= 2:
                    tot += e0.elapsed_time(e1)
            ms = tot / n_it
            tf = 2.0 * M * 4096 * 4096 / ms / 1e9
            out["weight_only_4096x4096_M%d_%s" % (M, name)] = {
                "us": ms * 1e3, "TFLOP/s": tf, "frac_bf16_burst": tf / peaks["bf16_burst"]}
            # the same with the weights prepacked once, outside the call
            pre = mxp.mxp_gemm_prepack(pw, True)
            tot = 0.0
            for i in range(n_it + 2):
                flush.fill_(i & 255)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                mxp.mxp_gemm_dense_prepacked(a, pw, pre, out=d, workspace=ws)
                e1.record()
                torch.cuda.synchronize()
                if i >= 2:
                    tot += e0.elapsed_time(e1)
            ms = tot / n_it
            tf = 2.0 * M * 4096 * 4096 / ms / 1e9
            out["weight_only_4096x4096_M%d_%s_prepacked" % (M, name)] = {
                "us": ms * 1e3, "TFLOP/s": tf, "frac_bf16_burst": tf / peaks["bf16_burst"]}
            del pw, ws, pre
        del a, w, d
    del flush
    return out


def part_prefill(mxp, synth, peaks, iters):
    import torch
    out = {}
    fp4_burst = peaks["bf16_burst"] * NOMINAL_FP4_OVER_BF16
    # ---- config 4: prefill GEMM on packed operands, every mode pair
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for cfg, (a_bits, w_bits), n_it in (("cfg4", synth.config4(), iters),
                                        ("cfg5", synth.config5(), max(1, iters // 3))):
        a, w = dev_bf16(a_bits), dev_bf16(w_bits)
        del a_bits, w_bits
        M, K = a.shape
        N = w.shape[0]
        d = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros(max(4096, mxp.mxp_gemm_workspace_bytes(M, N, K, False, 1, 1)),
                         dtype=torch.uint8, device="cuda")
        for an, am in (("mxfp4", 0), ("mxfp4+", 1)):
            for bn, bm in (("mxfp4", 0), ("mxfp4+", 1)):
                pa, pw = mxp.mxp_quantize(a, am), mxp.mxp_quantize(w, bm)
                tot = 0.0
                for i in range(n_it + 2):
                    flush.fill_(i & 255)  # evict L2 between timed launches
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    mxp.mxp_gemm(pa, pw, out=d, workspace=ws)
                    e1.record()
                    torch.cuda.synchronize()
                    if i >= 2:
                        tot += e0.elapsed_time(e1)
                ms = tot / n_it
                tf = 2.0 * M * N * K / ms / 1e9
                out["prefill_%s_A-%s_W-%s" % (cfg, an, bn)] = {
                    "us": ms * 1e3, "TFLOP/s": tf, "frac_fp4_peak_4x_bf16_burst": tf / fp4_burst,
                    "frac_fp4_nominal_9PF": tf / 9000.0}
                try:  # the GEMM kernel's own cycle / nanosecond stamps (last launch)
                    cyc, ns = mxp.mxp_gemm_clock_stamp(ws)
                    macs = 8192 if (am or bm) else 16384  # per SM per clock: 8-bit containers, FP4
                    sms = torch.cuda.get_device_properties(0).multi_processor_count
                    out["prefill_%s_A-%s_W-%s" % (cfg, an, bn)].update({
                        "kernel_us": ns / 1e3, "sm_mhz_in_kernel": cyc / ns * 1e3,
                        "tensor_pipe_util_at_that_clock": 2.0 * M * N * K / (cyc * sms * 2 * macs)})
                except mxp.MxpError:
                    pass
                del pa, pw
        if cfg == "cfg5":   # MX++ on both sides: same kernel, delta handled by the prepack
            pa, pw = mxp.mxp_quantize(a, mxp.MODE_MXFP4_PP), mxp.mxp_quantize(w, mxp.MODE_MXFP4_PP)
            tot = 0.0
            for i in range(n_it + 2):
                flush.fill_(i & 255)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                mxp.mxp_gemm(pa, pw, out=d, workspace=ws)
                e1.record()
                torch.cuda.synchronize()
                if i >= 2:
                    tot += e0.elapsed_time(e1)
            ms = tot / n_it
            tf = 2.0 * M * N * K / ms / 1e9
            out["prefill_cfg5_A-mxfp4++_W-mxfp4++"] = {
                "us": ms * 1e3, "TFLOP/s": tf, "frac_fp4_peak_4x_bf16_burst": tf / fp4_burst,
                "frac_fp4_nominal_9PF": tf / 9000.0}
            del pa, pw
            # MXFP6 / MXFP6+ operands (E2M3 elements; an MXFP6+ operand costs a second pass) and
            # MXFP8 operands (E4M3 elements, read as stored; an MXFP8+ operand costs three passes)
            for an, am, bn, bm in (("mxfp6", mxp.MODE_MXFP6, "mxfp6", mxp.MODE_MXFP6),
                                   ("mxfp6+", mxp.MODE_MXFP6_PLUS, "mxfp6", mxp.MODE_MXFP6),
                                   ("mxfp6+", mxp.MODE_MXFP6_PLUS, "mxfp4", mxp.MODE_MXFP4),
                                   ("mxfp8", mxp.MODE_MXFP8, "mxfp8", mxp.MODE_MXFP8),
                                   ("mxfp8", mxp.MODE_MXFP8, "mxfp4+", mxp.MODE_MXFP4_PLUS),
                                   ("mxfp8+", mxp.MODE_MXFP8_PLUS, "mxfp8", mxp.MODE_MXFP8)):
                ws6 = torch.zeros(mxp.mxp_gemm_workspace_bytes(M, N, K, False, am, bm),
                                  dtype=torch.uint8, device="cuda")
                pa, pw = mxp.mxp_quantize(a, am), mxp.mxp_quantize(w, bm)
                tot = 0.0
                for i in range(n_it + 2):
                    flush.fill_(i & 255)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    mxp.mxp_gemm(pa, pw, out=d, workspace=ws6)
                    e1.record()
                    torch.cuda.synchronize()
                    if i >= 2:
                        tot += e0.elapsed_time(e1)
                ms = tot / n_it
                tf = 2.0 * M * N * K / ms / 1e9
                out["prefill_cfg5_A-%s_W-%s" % (an, bn)] = {
                    "us": ms * 1e3, "TFLOP/s": tf, "frac_fp4_peak_4x_bf16_burst": tf / fp4_burst,
                    "frac_fp4_nominal_9PF": tf / 9000.0}
                del pa, pw, ws6
        del a, w, d, ws
        torch.cuda.empty_cache()
    return out



def _r(x, n=4):
    """Rounded to n significant digits (keeps the JSON line short)."""
    return float("%.*g" % (n, x)) if isinstance(x, float) else x


def timed_flushed(fn, n_it, flush, pre=2):
    """Mean milliseconds of `fn`, one launch at a time, L2 evicted before each."""
    import torch
    tot = 0.0
    for i in range(n_it + pre):
        flush.fill_(i & 255)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        if i >= pre:
            tot += e0.elapsed_time(e1)
    return tot / n_it


def timed_queued(fn, n_it, flush):
    """Mean milliseconds of `fn` with cold L2 and without the host's launch latency: n_it times
    (evict L2, fn) queued back to back, minus the same queue of evictions alone.  This is what a
    call costs inside a stream that the host keeps ahead of, or inside a CUDA graph."""
    import torch

    def queue(with_fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(n_it):
            flush.fill_(i & 255)
            if with_fn:
                fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n_it
    for _ in range(2):
        fn()
    queue(True)
    return queue(True) - queue(False)


def graph_of(run, n=8):
    """CUDA graph of n back-to-back calls of `run` (warmed up on a side stream first)."""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(n):
            run()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(n):
            run()
    return g


def targets(mxp, synth, peaks):
    """The scorecard: every configuration's kernel against its roofline, MXFP4+ beside plain
    MXFP4, in a form short enough to survive at the end of the JSON line.
      quantize (config 2) and decode (config 3): fraction of the measured HBM copy bandwidth;
      prefill (configs 4 and 5): fraction of the dense FP4 peak = 4 x measured bf16 burst rate.
    One launch (or one graph of 32 chained calls) at a time with cold L2, i.e. the burst power state."""
    import torch
    hbm = peaks["hbm_gbs"]
    fp4 = peaks["bf16_burst"] * NOMINAL_FP4_OVER_BF16
    out = {"denominators": {"hbm_GBs": hbm, "fp4_TFLOPs": fp4,
                            "note": "%s copy bandwidth; 4 x %s bf16 burst" % (peaks["src"], peaks["src"])}}
    MX, MXP = mxp.MODE_MXFP4, mxp.MODE_MXFP4_PLUS
    # ---- config 2: quantize 8192 x 8192 bf16
    x = dev_bf16(synth.config2())
    q = {}
    for name, mode in (("mx+", MXP), ("mxfp4", MX)):
        buf = mxp.alloc_packed(x.shape[0], x.shape[1], mode, index_for_mxfp4=False)
        ms = time_loop(lambda: mxp.mxp_quantize(x, mode, out=buf), 20)
        nbytes = x.numel() * (2 + 0.5 + 1 / 32 + (1 / 32 if mode == MXP else 0))
        q[name] = {"us": _r(ms * 1e3), "GBs": _r(nbytes / ms / 1e6), "frac": _r(nbytes / ms / 1e6 / hbm, 3)}
    q["mx+/mxfp4"] = _r(q["mx+"]["us"] / q["mxfp4"]["us"], 3)
    out["quantize_cfg2"] = q
    del x
    # ---- config 3: decode GEMM, eight rotating weight copies (> L2), graphs of 32 launches (a
    # token's pass over a model's layers is hundreds of such calls in one graph; the first call of
    # a graph cannot overlap the graph before it, and with eight calls per graph that boundary
    # alone adds ~0.5 us to every call's average).
    kChain = 32
    # "tc": weights re-tiled once, FP4 tensor path (mxp_gemm_decode_prepacked_next: each call
    # names the weights of the next; "tc_nohint": mxp_gemm_decode_prepacked, without); "reg": the
    # streamed register-decode kernel behind mxp_gemm; both as chains of programmatic dependents
    # (constant weights), which is what a captured decode loop can use.
    a16, w_bits = synth.config3(16)
    w = dev_bf16(w_bits)
    N, K = w.shape
    dec = {}
    for name, mode in (("mx+", MXP), ("mxfp4", MX)):
        packed = [mxp.mxp_quantize(w, mode) for _ in range(8)]
        tiled = [mxp.mxp_gemm_decode_prepack(p) for p in packed]
        wbytes = N * K * (0.5 + 1 / 32 + (1 / 32 if mode == MXP else 0))
        row = {}
        for M in (1, 8, 16):
            a = dev_bf16(a16[:M].copy())
            d = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            ws = torch.zeros(max(256, mxp.mxp_gemm_decode_workspace_bytes(M, K)), dtype=torch.uint8, device="cuda")
            st = {"i": 0}
            tot = wbytes + M * K * 2 + M * N * 2

            def run_tc():  # every call names the next one's weights, as a decoder knows its next layer
                mxp.mxp_gemm_decode_prepacked(a, tiled[st["i"] % 8], out=d, workspace=ws, chained=True,
                                              next_w=tiled[(st["i"] + 1) % 8])
                st["i"] += 1

            def run_tc_nohint():
                mxp.mxp_gemm_decode_prepacked(a, tiled[st["i"] % 8], out=d, workspace=ws, chained=True)
                st["i"] += 1

            def run_reg():
                mxp.mxp_gemm_decode_chained(a, packed[st["i"] % 8], d)
                st["i"] += 1
            us_tc = time_loop(graph_of(run_tc, kChain).replay, 6, warmup=2) / kChain * 1e3
            us_nh = time_loop(graph_of(run_tc_nohint, kChain).replay, 6, warmup=2) / kChain * 1e3
            us_reg = time_loop(graph_of(run_reg, kChain).replay, 6, warmup=2) / kChain * 1e3
            row["M%d" % M] = {"tc_us": _r(us_tc), "tc_nohint_us": _r(us_nh), "reg_us": _r(us_reg),
                              "frac": _r(tot / min(us_tc, us_nh, us_reg) / 1e3 / hbm, 3)}
        dec[name] = row
        del packed, tiled
    best = lambda e: min(e["tc_us"], e["tc_nohint_us"], e["reg_us"])
    dec["mx+/mxfp4_M1"] = _r(best(dec["mx+"]["M1"]) / best(dec["mxfp4"]["M1"]), 3)
    out["decode_cfg3"] = dec
    del w
    # ---- the same at M = 1 on a larger weight matrix (14336 x 4096, an 8B model's MLP width):
    # the part of a call that carries no weight traffic weighs less.  Not one of the configs:
    # beside them for context, the goal below is judged on config 3.
    big = {}
    N2, K2 = 14336, 4096
    a2_bits, w2_bits = synth.config3(1, N2, K2, seed=11)
    a2, w2 = dev_bf16(a2_bits), dev_bf16(w2_bits)
    for name, mode in (("mx+", MXP), ("mxfp4", MX)):
        tiled = [mxp.mxp_gemm_decode_prepack(mxp.mxp_quantize(w2, mode)) for _ in range(8)]
        d = torch.empty((1, N2), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros(max(256, mxp.mxp_gemm_decode_workspace_bytes(1, K2)), dtype=torch.uint8, device="cuda")
        st = {"i": 0}

        def run_big():
            mxp.mxp_gemm_decode_prepacked(a2, tiled[st["i"] % 8], out=d, workspace=ws, chained=True,
                                          next_w=tiled[(st["i"] + 1) % 8])
            st["i"] += 1
        us = time_loop(graph_of(run_big, kChain).replay, 6, warmup=2) / kChain * 1e3
        tot = N2 * K2 * (0.5 + 1 / 32 + (1 / 32 if mode == MXP else 0)) + K2 * 2 + N2 * 2
        big[name] = {"tc_us": _r(us), "frac": _r(tot / us / 1e3 / hbm, 3)}
        del tiled
    out["decode_14336x4096_M1"] = big
    del w2, a2
    # ---- configs 4 and 5: prefill.  Per mode pair the mxp_gemm_prepacked call (weights prepared
    # once; the activations' preparation is inside the timed call), queued behind an L2 eviction
    # (timed_queued: device time, not the host's launch latency).  One-sided pairs three ways:
    # S1 = FP4 main pass + sparse residual instruction (the default), S2 = one pass on widened
    # codes, eq4_dense = the in-place kernels with dense residual passes.
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for cfg, (a_bits, w_bits), n_it in (("cfg4", synth.config4(), 20), ("cfg5", synth.config5(), 4)):
        a, w = dev_bf16(a_bits), dev_bf16(w_bits)
        del a_bits, w_bits
        M, K = a.shape
        N = w.shape[0]
        fl = 2.0 * M * N * K
        d = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros(mxp.mxp_gemm_workspace_bytes(M, N, K, False, MXP, MXP), dtype=torch.uint8, device="cuda")
        small = torch.zeros(4096, dtype=torch.uint8, device="cuda")
        pf = {}
        qa = {m: mxp.mxp_quantize(a, m) for m in (MX, MXP)}
        qw = {m: mxp.mxp_quantize(w, m) for m in (MX, MXP)}
        for name, am, bm in (("plain", MX, MX), ("A+", MXP, MX), ("W+", MX, MXP), ("both", MXP, MXP)):
            pre = mxp.mxp_gemm_prepack(qw[bm], mxp.mxp_gemm_prepack_form(am, bm))
            ms = timed_queued(lambda: mxp.mxp_gemm_prepacked(qa[am], qw[bm], pre, out=d, workspace=ws), n_it, flush)
            cyc, ns = mxp.mxp_gemm_clock_stamp(ws)
            e = {"us": _r(ms * 1e3), "TFLOPs": _r(fl / ms / 1e9), "frac_fp4": _r(fl / ms / 1e9 / fp4, 3),
                 "kernel_us": _r(ns / 1e3), "kernel_mhz": int(cyc / ns * 1e3)}
            if name in ("A+", "W+"):
                mxp.mxp_debug_override(mxp.KNOB_ONE_SIDED, 1)
                try:
                    pre2 = mxp.mxp_gemm_prepack(qw[bm], mxp.mxp_gemm_prepack_form(am, bm))
                    ms2 = timed_queued(lambda: mxp.mxp_gemm_prepacked(qa[am], qw[bm], pre2, out=d, workspace=ws),
                                       n_it, flush)
                finally:
                    mxp.mxp_debug_override(mxp.KNOB_ONE_SIDED, 0)
                ms3 = timed_queued(lambda: mxp.mxp_gemm(qa[am], qw[bm], out=d, workspace=small), max(1, n_it // 2), flush)
                e.update({"S2_wide_us": _r(ms2 * 1e3), "eq4_dense_us": _r(ms3 * 1e3)})
                del pre2
            pf[name] = e
            del pre
        for name in ("A+", "W+", "both"):
            pf[name]["x_plain"] = _r(pf[name]["us"] / pf["plain"]["us"], 3)
        # the headline's own step on this shape: fused quantizer + GEMM on prepacked MXFP4+ weights
        pre = mxp.mxp_gemm_prepack(qw[MXP], mxp.PREPACK_WIDE)
        pa = mxp.alloc_packed(M, K, MXP)

        def step():
            mxp.mxp_quantize_gemm_ready(a, MXP, ws, out=pa)
            mxp.mxp_gemm_ready(pa, qw[MXP], pre, ws, out=d)
        ms = timed_queued(step, n_it, flush)
        pf["step_both"] = {"us": _r(ms * 1e3), "TFLOPs": _r(fl / ms / 1e9), "frac_fp4": _r(fl / ms / 1e9 / fp4, 3)}
        # the paper's main scenario as a step: activations to MXFP4+, split per Eq. 4 by the
        # quantizer itself, against MXFP4 weights prepared once (sparse residual GEMM): 2 launches
        pre_plain = mxp.mxp_gemm_prepack(qw[MX], mxp.PREPACK_PLAIN)

        def step_a_plus():
            mxp.mxp_quantize_gemm_ready(a, MXP, ws, out=pa, b_mode=MX)
            mxp.mxp_gemm_ready(pa, qw[MX], pre_plain, ws, out=d)
        ms = timed_queued(step_a_plus, n_it, flush)
        pf["step_A+"] = {"us": _r(ms * 1e3), "TFLOPs": _r(fl / ms / 1e9), "frac_fp4": _r(fl / ms / 1e9 / fp4, 3)}
        del pre_plain
        out["prefill_" + cfg] = pf
        del a, w, d, ws, qa, qw, pre, pa
        torch.cuda.empty_cache()
    del flush
    best_dec = min(out["decode_cfg3"][m]["M%d" % M_]["frac"] for m in ("mx+", "mxfp4") for M_ in (1, 8, 16))
    out["goals"] = {"quantize>=0.70_hbm": out["quantize_cfg2"]["mx+"]["frac"] >= 0.70,
                    "decode>=0.60_hbm": best_dec >= 0.60,   # every M of config 3, both formats
                    "decode_M1>=0.60_hbm": {m: out["decode_cfg3"][m]["M1"]["frac"] >= 0.60 for m in ("mxfp4", "mx+")},
                    "prefill_mx+>=0.50_fp4": out["prefill_cfg5"]["A+"]["frac_fp4"] >= 0.50,
                    "prefill_both>=0.50_fp4": out["prefill_cfg5"]["both"]["frac_fp4"] >= 0.50,
                    "mx+_within_1.15x_plain": {"quantize": out["quantize_cfg2"]["mx+/mxfp4"] <= 1.15,
                                               "decode_M1": out["decode_cfg3"]["mx+/mxfp4_M1"] <= 1.15,
                                               "prefill_A+": out["prefill_cfg5"]["A+"]["x_plain"] <= 1.15}}
    return out


def sustained_probe(mxp, kind, seconds=2.0, iters=100000):
    """Issue-only tensor-core rate held for `seconds`: back-to-back probe launches, the mean of
    those in the second half (the board has settled to its power limit by then)."""
    rates = []
    t0 = time.perf_counter()
    while time.perf_counter() - t0 < seconds:
        pms, pfl = mxp.mxp_tensor_peak_probe(kind, iters)
        rates.append((time.perf_counter() - t0, pfl / pms / 1e9))
    late = [r for t, r in rates if t >= seconds / 2] or [r for _, r in rates]
    return sum(late) / len(late)


def run_ours(args, M, N, K, label):
    import torch
    import torch.distributed as dist
    from paper_2510_14557_b200 import build
    build.build()
    import paper_2510_14557_b200 as mxp
    from paper_2510_14557_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    peaks = measured_peaks()

    # synthetic operands (every rank: same weights, its own activation batch)
    a_bits = synth.f32_to_bf16_bits(synth.activations_normal(M, K, 4 + 1000 * rank, 0.01, 30.0))
    w_bits = synth.f32_to_bf16_bits(synth.weights(N, K, 104))
    a_host = torch.from_numpy(a_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    a_dev = a_host.cuda()
    w_dev = dev_bf16(w_bits)
    pw = mxp.mxp_quantize(w_dev, mxp.MODE_MXFP4_PLUS)   # weights are quantized once, offline,
    w_pre = mxp.mxp_gemm_prepack(pw, True)              # and prepared for the GEMM once
    del w_dev, w_bits
    pa = mxp.alloc_packed(M, K, mxp.MODE_MXFP4_PLUS)
    d_dev = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    d_host = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    ws = torch.zeros(max(4096, mxp.mxp_gemm_workspace_bytes(M, N, K, False, 1, 1)),
                     dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    # One step = two launches: the quantizer (packed MXFP4+ planes of the activations plus their
    # GEMM-ready form, written into the GEMM's workspace) and the GEMM.
    def step(ev=None):
        mxp.mxp_quantize_gemm_ready(a_dev, mxp.MODE_MXFP4_PLUS, ws, out=pa)
        if ev is not None:
            ev[0].record(stream)
        mxp.mxp_gemm_ready(pa, pw, w_pre, ws, out=d_dev)
        if ev is not None:
            ev[1].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing.  The warm-up runs straight into the timed region (only the
    # barrier in between): this board lowers its clocks a few tens of milliseconds into a dense
    # load, and a pause would let it recover (the default warm-up is long enough to get there).
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    warm0, warm1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    warm0.record(stream)
    for _ in range(max(3, args.warmup)):
        step()
    warm1.record(stream)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(kev[i])
    e1.record(stream)
    barrier()
    if mxp.mxp_gemm_status(ws) != 0:
        raise RuntimeError("mxp_gemm reported a device-side timeout")
    ms_local = e0.elapsed_time(e1) / args.steps
    busy_ms = warm0.elapsed_time(warm1) + e0.elapsed_time(e1)  # dense load up to the end of timing
    time.sleep(0.03)                       # let the sampler's last line of the timed region arrive
    timed_samples = len(sampler.lines)
    # SM cycles and nanoseconds the last timed step's GEMM kernel ran for, stamped by the kernel itself
    stamp_cycles, stamp_ns = mxp.mxp_gemm_clock_stamp(ws)
    # ---- the settled state, whatever --steps was: this board lowers its clocks a few tens of
    # milliseconds into a dense tensor load, so keep stepping (no pause) until at least 300 ms of
    # dense load lie behind, then time 40 more steps.
    sus = None
    if world == 1:
        n_fill = max(0, int((300.0 - busy_ms) / max(ms_local, 1e-3)) + 1)
        for _ in range(n_fill):
            step()
        s_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(40)]
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        n_before = len(sampler.lines)
        s0.record(stream)
        for i in range(40):
            step(s_ev[i])
        s1.record(stream)
        torch.cuda.synchronize()
        time.sleep(0.05)
        sus_lines = sampler.lines[n_before:]
        sus_ms = s0.elapsed_time(s1) / 40
        sus_gemm_ms = sum(a.elapsed_time(b) for a, b in s_ev) / 40
        sus_cycles, sus_ns = mxp.mxp_gemm_clock_stamp(ws)
        sus_mhz = []
        for ln in sus_lines:
            f = [x.strip() for x in ln.split(",")]
            try:
                sus_mhz.append(float(f[1]))
            except (ValueError, IndexError):
                pass
        sus = {"after_ms_of_dense_load": round(busy_ms + n_fill * ms_local, 1), "steps": 40,
               "ms_per_step": sus_ms, "value": 2.0 * M * N * K / sus_ms / 1e9, "unit": UNIT,
               "gemm_kernel_ms": sus_gemm_ms, "gemm_TFLOPs": 2.0 * M * N * K / sus_gemm_ms / 1e9,
               "sm_mhz_sampled": statistics.median(sus_mhz) if sus_mhz else None,
               "sm_mhz_in_kernel": sus_cycles / sus_ns * 1e3}
    clocks = sampler.stop(upto=timed_samples) if rank == 0 else None
    gemm_ms = sum(a.elapsed_time(b) for a, b in kev) / args.steps
    flops_step = 2.0 * M * N * K
    ms, flops_all = aggregate(ms_local, flops_step, dist if world > 1 else None)

    # ---- end to end: pinned host activations in, result matrix out, every step.  Copies and
    # compute run on three streams with two sets of buffers, so the input copy of step i + 1
    # and the output copy of step i - 1 overlap the kernels of step i (every step still copies
    # its whole input in and its whole result out inside the timed region).
    a_dev2 = torch.empty_like(a_dev)
    pa2 = mxp.alloc_packed(M, K, mxp.MODE_MXFP4_PLUS)
    d_dev2 = torch.empty_like(d_dev)
    d_host2 = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    bufs = [(a_dev, pa, d_dev, d_host), (a_dev2, pa2, d_dev2, d_host2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        a_d, p_a, d_d, d_h = bufs[i % 2]
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_cmp[i % 2])   # step i - 2 has read this input buffer
            a_d.copy_(a_host, non_blocking=True)
            ev_in[i % 2].record(s_in)
        stream.wait_event(ev_in[i % 2])
        if i >= 2:
            stream.wait_event(ev_out[i % 2])     # step i - 2's result has left this buffer
        mxp.mxp_quantize_gemm_ready(a_d, mxp.MODE_MXFP4_PLUS, ws, out=p_a)
        mxp.mxp_gemm_ready(p_a, pw, w_pre, ws, out=d_d)
        ev_cmp[i % 2].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[i % 2])
            d_h.copy_(d_d, non_blocking=True)
            ev_out[i % 2].record(s_out)

    for i in range(2):
        e2e_step(i)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(4, min(args.steps, 8))
    e2.record(stream)
    s_in.wait_event(e2)
    for i in range(e2e_steps):
        e2e_step(i + 2)
    e3.record(s_out)
    barrier()
    e2e_ms, e2e_flops = aggregate(e2.elapsed_time(e3) / e2e_steps, flops_step, dist if world > 1 else None)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # The roofline is the one the metric names: the dense FP4 tensor peak, 4 x the measured bf16
    # rate (nominal FP4 : bf16 ratio), burst figure, whatever the run's length -- the settled
    # state has its own record (`sustained`, against 4 x the sustained bf16 figure).  The step
    # with two MX+ operands runs one kind::mxf8f6f4 pass on operands widened to E2M3 codes, whose
    # instruction rate is half the FP4 rate: the fraction of that ceiling is printed beside.
    fp4_burst = peaks["bf16_burst"] * NOMINAL_FP4_OVER_BF16
    fp4_sustained = peaks["bf16_sustained"] * NOMINAL_FP4_OVER_BF16
    achieved = flops_step / gemm_ms / 1e9
    if sus is not None:
        sus["frac_of_fp4_sustained_peak"] = sus["gemm_TFLOPs"] / fp4_sustained
        sus["frac_of_8bit_kind_sustained_peak"] = sus["gemm_TFLOPs"] / (peaks["bf16_sustained"] * NOMINAL_FP8_OVER_BF16)
        sus["peak"] = "4 x %s bf16 sustained = %.0f TFLOP/s" % (peaks["src"], fp4_sustained)
    # issue-only tcgen05 rates on this device (operands resident in shared memory): a burst of a
    # few milliseconds and, for the two dense kinds, the rate held over two seconds
    probes = {}
    for name, kind in (("mxf4", 0), ("mxf8f6f4", 1), ("mxf4_plus_sparse_residual", 5)):
        try:
            pms, pfl = mxp.mxp_tensor_peak_probe(kind, 20000)
            probes[name] = _r(pfl / pms / 1e9)
        except Exception:
            probes[name] = None
    if world == 1:
        for name, kind in (("mxf4_sustained_2s", 0), ("mxf8f6f4_sustained_2s", 1)):
            try:
                probes[name] = _r(sustained_probe(mxp, kind))
            except Exception:
                probes[name] = None
    # The board's power limit, not the tensor pipe, sets the SM clock of a dense GEMM: the kernel's
    # own cycle and nanosecond stamps give the clock it really ran at, and the share of the tensor
    # pipe's rate AT THAT CLOCK (nominal 8192 8-bit-container MACs per SM per clock) it used.
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    in_kernel_mhz = stamp_cycles / stamp_ns * 1e3
    kernel_only_tflops = flops_step / stamp_ns / 1e3
    pipe_tflops_at_clock = sms * 2 * 8192 * in_kernel_mhz * 1e6 / 1e12
    line = {
        "metric": METRIC, "value": flops_all / ms / 1e9, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "e2m3 codes holding E2M1/E0M3 values (kind::mxf8f6f4), fp32 accumulate",
        "data": "synthetic",
        "config": {"workload": label, "M": M, "N": N, "K": K, "a_mode": "MXFP4+", "w_mode": "MXFP4+",
                   "weights": "quantized and prepacked (mxp_gemm_prepack) once, outside the step",
                   "out": "bf16", "l2": "inputs larger than L2 (no flush needed)" if (M * K * 2 + N * K // 2) > (126 << 20)
                   else "inputs smaller than L2: numbers include L2 hits"},
        "roofline": {"bound": "tensor", "kernel": "mxp_gemm_ready = gemm_tc_stream_kernel<wide, 2 halves>",
                     "achieved": achieved, "peak": fp4_burst,
                     "unit": "TFLOP/s", "frac": achieved / fp4_burst, "traffic": NCU_DRAM_TRAFFIC.get(args.workload),
                     "peak_source": "dense FP4 peak = 4 x %s bf16 burst (nominal FP4 : bf16 ratio); %.0f ms of "
                                    "dense load up to the end of the timed region" % (peaks["src"], busy_ms),
                     "frac_of_fp4_sustained_peak": achieved / fp4_sustained,
                     "frac_of_8bit_kind_peak": achieved / (peaks["bf16_burst"] * NOMINAL_FP8_OVER_BF16),
                     "frac_of_fp4_nominal_9PF": achieved / 9000.0,
                     "kernel_ms": gemm_ms,
                     "issue_probe_tflops": probes,
                     "in_kernel": {"sm_mhz": in_kernel_mhz, "kernel_us": stamp_ns / 1e3,
                                   "tflops": kernel_only_tflops,
                                   "tensor_pipe_tflops_at_that_clock": pipe_tflops_at_clock,
                                   "tensor_pipe_util": kernel_only_tflops / pipe_tflops_at_clock}},
        "e2e": {"value": e2e_flops / e2e_ms / 1e9, "unit": UNIT, "h2d_bytes_per_step": M * K * 2,
                "d2h_bytes_per_step": M * N * 2, "ms_per_step": e2e_ms},
        "gpu_launches": 2 * args.steps,  # quantize (with the GEMM-ready planes), GEMM
        "clocks": clocks,
    }
    if world == 1:
        line["cpu_baseline"] = cpu_baseline(M, N, K)
        del d_dev, d_host, pa, pw, a_dev, w_pre, ws, bufs, a_dev2, pa2, d_dev2, d_host2
        torch.cuda.empty_cache()
        if args.parts:
            try:
                line["parts"] = parts(mxp, synth, peaks)
            except Exception as e:  # report, never hide
                line["parts"] = {"error": repr(e)}
        # the last two keys, so that they survive at the end of the line
        line["sustained"] = sus
        if not args.no_targets:
            try:
                line["targets"] = targets(mxp, synth, peaks)
            except Exception as e:
                line["targets"] = {"error": repr(e)}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=60)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=sorted(WORKLOADS))
    ap.add_argument("--no-targets", action="store_true", help="skip the per-configuration scorecard")
    ap.add_argument("--parts", action="store_true", help="add the long per-kernel list")
    ap.add_argument("--no-parts", action="store_true",
                    help="the step only: same as --no-targets (the flag's older name)")
    ap.add_argument("--only", default=None,
                    choices=["quantize", "decode", "prefill", "prefill_cfg4", "decode_tc"],
                    help="run one per-config part only and print its numbers (profiler captures)")
    ap.add_argument("--iters-scale", type=float, default=1.0)
    args = ap.parse_args()
    M, N, K, label = WORKLOADS[args.workload]
    if args.no_parts:
        args.no_targets = True
    if args.only is not None:
        from paper_2510_14557_b200 import build, synth
        build.build()
        import paper_2510_14557_b200 as mxp
        print(json.dumps({"parts": parts(mxp, synth, measured_peaks(), args.only, args.iters_scale)}))
    elif args.impl == "reference":
        run_reference(args, M, N, K, label)
    else:
        run_ours(args, M, N, K, label)


if __name__ == "__main__":
    main()
