#!/usr/bin/env python
"""Benchmark of the W4A8 quantized linear (Sec. 3.4) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--no-sweep] [--impl reference]

One "step" is one pass of the whole hot path - quantise the activations, then the W4A8
matrix multiply - over one batch of the speculative-verify configuration (M = 8 draft tokens,
K = 4096, N = 6144; Sec. 3.2), through w4a8_linear (two kernels chained with programmatic
dependent launch).  The weights are packed once beforehand (they are quantised offline, Sec. 3.4).
That configuration is memory-bound, so the metric is HBM GB/s: algorithmic bytes of the
step divided by time.  Successive steps use different packed copies of the layer (more
than two L2 capacities in total), so weights always come from HBM, as they do in a decoder
that walks through dozens of distinct layers.  The timed region is one CUDA-graph launch of
exactly K steps, bracketed by CUDA events, a barrier and a device synchronise.

Printed on one JSON line: the step throughput (`value`), the same measured end to end from
pinned host buffers through w4a8_linear_host (`e2e`), the roofline of the dominant kernel
(`roofline`), the CPU oracle timed on this host's cores (`cpu_baseline`), the SM clocks seen
during the timed region (`clocks`), and - unless --no-sweep - TOPS / GB/s / roofline fraction
for all four linears of the decoder layer at M = 1...4096 (`sweep`) and the four linears of one layer
chained in one graph (`layer_chain`).

Multi-GPU: the path does not shard (one GPU per model replica); with --gpus N every rank
runs the same replica on its own GPU and the value is the sum over ranks (weak scaling).
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_12932_b200 import workload as wl  # noqa: E402

HEADLINE = "spec_verify"
METRIC = "w4a8_linear_hbm_gbs"
NOMINAL_HBM_GBS = 8000.0          # "~8 TB/s"
NOMINAL_INT8_TOPS = 4500.0        # dense INT8, twice the nominal dense bf16 rate
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
L2_BYTES_ASSUMED = 126 * 2 ** 20


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS,
                bf16_tflops_sustained=1400.0, source="fallback")


def measure_int8_peak(torch, seconds=2.0):
    """A library INT8 GEMM (torch._int_mm, 8192^3) timed on this GPU: best single launch (burst) and a back-to-back
    loop of `seconds` (sustained, under the power cap).  Timing a library is allowed; it is not on the product path."""
    try:
        n = 8192
        a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device="cuda")
        b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device="cuda")
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = 1e9
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(seconds * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch._int_mm(a, b)
        e1.record()
        e1.synchronize()
        sustained = e0.elapsed_time(e1) / reps
        ops = 2.0 * n ** 3
        del a, b
        torch.cuda.empty_cache()
        return {"int8_tops_burst": ops / best / 1e9, "int8_tops_sustained": ops / sustained / 1e9,
                "how": f"torch._int_mm {n}^3, best of 10 and {reps} back to back"}
    except Exception as ex:      # noqa: BLE001 - the library routine may be missing; the stand-in is then used alone
        return {"int8_tops_burst": None, "int8_tops_sustained": None, "how": f"unavailable: {type(ex).__name__}"}


def step_bytes(M, N, K):
    return wl.algorithmic_bytes_quantize(M, K) + wl.algorithmic_bytes_gemm(M, N, K)


# ----------------------------------------------------------------------------- clocks ----
class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, f"/tmp/w4a8_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=self.out, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                t = [v.strip() for v in line.split(",")]
                if len(t) < 7:
                    continue
                try:
                    sm.append(float(t[0])), smax.append(float(t[1]))
                except ValueError:
                    continue
                for n, v in zip(names, t[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "samples": len(sm),
                "reasons": sorted(reasons)}


def workload_name(M, N, K):
    return f"{HEADLINE}: M={M} K={K} N={N} group=128; step = w4a8_linear (w4a8_quantize_act + w4a8_gemm)"


# ----------------------------------------------------------------------- CPU oracle arm ---
def time_oracle(case, min_seconds, max_steps=None):
    """The CPU oracle, as it stands, on the whole headline step; returns (steps, seconds, threads)."""
    from oracle import cfast
    cfast.build()
    cfast.w4a8_linear(case["x"], case["qw"], case["sw"], case["z"], case["group"])     # page in
    steps, t0 = 0, time.perf_counter()
    while True:
        cfast.w4a8_linear(case["x"], case["qw"], case["sw"], case["z"], case["group"])
        steps += 1
        el = time.perf_counter() - t0
        if (max_steps is not None and steps >= max_steps) or (max_steps is None and el >= min_seconds):
            return steps, el, cfast.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    case = wl.make_config(HEADLINE)
    M, N, K = case["M"], case["N"], case["K"]
    time_oracle(case, 0.0, max_steps=max(args.warmup, 1))
    steps, el, threads = time_oracle(case, 0.0, max_steps=args.steps)
    gbs = step_bytes(M, N, K) * steps / el / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": el / steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8 x uint4 -> int32, fp64 scaling", "data": "synthetic",
        "config": {"workload": workload_name(M, N, K)},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                         "sample": f"the whole step, {steps} repetitions"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------ GPU arm ---
def to_dev16(torch, a, dtype):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(dtype)


class Timer:
    def __init__(self, torch):
        self.torch = torch

    def graph_ms(self, fn, replays=1, warm=3):
        """Capture fn() into a CUDA graph, replay it; returns best and median ms per replay."""
        torch = self.torch
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            fn()                                   # eager warm-up (sets function attributes before capture)
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        for _ in range(warm):
            g.replay()
        torch.cuda.synchronize()
        times = []
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        return g, times


def max_over_ranks(ms, dist, device):
    """A time measured on every rank -> the slowest rank's (what a replicated job waits for)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_step, steps, world, ms):
    """Replicas only: every rank runs the same steps on its own GPU; the job's throughput is the sum."""
    return bytes_per_step * steps * world / (ms * 1e-3) / 1e9


def copies_for(nbytes, l2_bytes):
    return int(np.ceil(2.0 * l2_bytes / nbytes)) + 1


def run_sweep(torch, B, peaks, l2_bytes, timer):
    """All four linears at every M of the sweep: GEMM alone, rotating cold weight copies; best of 5 graph replays.
    frac_measured: against the measured HBM copy rate / 2 x the measured bf16 rate; frac_int8_mm: against the library
    INT8 GEMM measured in this run (burst)."""
    out, out_pc = [], []
    int8_peak = 2.0 * peaks["bf16_tflops"]
    int8_mm = peaks.get("int8_tops_burst")
    for lname, (K, N) in wl.LAYERS.items():
        case = wl.make_sweep_layer(lname)
        qw = torch.from_numpy(case["qw"]).cuda()
        sw = to_dev16(torch, case["sw"], torch.float16)
        z = torch.from_numpy(case["z"]).cuda()
        packed0 = B.w4a8_pack_weights(qw, sw, z)
        ncopies = copies_for(packed0.numel(), l2_bytes)
        packed = [packed0] + [packed0.clone() for _ in range(ncopies - 1)]
        del qw, sw, z
        ws = B.new_workspace(max(wl.SWEEP_M), N, K)
        x_all = to_dev16(torch, case["x"], torch.bfloat16)
        for M in wl.SWEEP_M:
            qa, sa, asum = B.w4a8_quantize_act(x_all[:M].contiguous())
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            reps = 2 if M >= 1024 else 4

            B.w4a8_gemm(qa, sa, asum, packed[0], N, ws, out=y)
            B.w4a8_check_status(ws)

            def body():
                for _ in range(reps):
                    for p in packed:
                        B.w4a8_gemm(qa, sa, asum, p, N, ws, out=y)
            _, times = timer.graph_ms(body, replays=5, warm=2)
            B.w4a8_check_status(ws)
            us = min(times) * 1e3 / (reps * ncopies)
            ops, nbytes = wl.algorithmic_ops(M, N, K), wl.algorithmic_bytes_gemm(M, N, K)
            t_c_meas, t_m_meas = ops / (int8_peak * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)
            t_c_nom, t_m_nom = ops / (NOMINAL_INT8_TOPS * 1e12), nbytes / (NOMINAL_HBM_GBS * 1e9)
            out.append({"layer": lname, "M": M, "us": round(us, 2),
                        "tops": round(ops / us / 1e6, 1), "gbs": round(nbytes / us / 1e3, 1),
                        "bound": "int8" if t_c_meas > t_m_meas else "hbm",
                        "frac_measured": round(max(t_c_meas, t_m_meas) * 1e6 / us, 3),
                        "frac_nominal": round(max(t_c_nom, t_m_nom) * 1e6 / us, 3),
                        "frac_int8_mm": (round(max(ops / (int8_mm * 1e12), t_m_meas) * 1e6 / us, 3) if int8_mm else None),
                        "kernel": plan_name(B, M, N, K)})
            if M >= 1024:
                # the same pipeline with one drain per tile (w4a8_gemm_per_channel: scales constant along K;
                # it reads the first group's scales only, so the timing needs no second set of weights)
                def body_pc():
                    for _ in range(reps):
                        for p in packed:
                            B.w4a8_gemm_per_channel(qa, sa, p, N, ws, out=y)
                _, times = timer.graph_ms(body_pc, replays=5, warm=2)
                B.w4a8_check_status(ws)
                us = min(times) * 1e3 / (reps * ncopies)
                out_pc.append({"layer": lname, "M": M, "us": round(us, 2), "tops": round(ops / us / 1e6, 1),
                               "frac_measured": round(max(t_c_meas, t_m_meas) * 1e6 / us, 3),
                               "frac_nominal": round(max(t_c_nom, t_m_nom) * 1e6 / us, 3)})
        del packed, packed0, x_all
        torch.cuda.empty_cache()
    return out, out_pc


def plan_name(B, M, N, K):
    """The kernel w4a8_gemm launches for a size, from the library's own planner."""
    p = B.w4a8_plan(M, N, K)
    if p["family"] == B.PATH_STRIP:
        return f"gemm_strip_kernel<{p['tile_m'] // 8},{p['strip_rows'] // 16}> x {p['ctas']} CTAs"
    if p["family"] == B.PATH_SPLITK:
        return f"gemm_cluster_kernel<{p['tile_m'] // 8}> x {p['ctas']} CTAs, {p['k_slices']} K slices"
    return (f"gemm_tcgen05_kernel<{p['tile_m']}> x {p['ctas']} CTAs" + (f", {p['k_slices']} K slices" if p["k_slices"] > 1 else "")
            + (", balanced walk" if p["balanced"] else ""))


def run_large_m_roofline(torch, B, peaks, l2_bytes, timer):
    """The tensor-core kernel alone on the streaming-prefill configuration (M = 1024, K = 4096, N = 24576: fused gate+up),
    cold weight copies in turn, median of 5 graph replays."""
    c = wl.CONFIGS["prefill_gate_up"]
    M, K, N = c["M"], c["K"], c["N"]
    rng = np.random.default_rng(11)
    r = wl.random_codes(rng, M, N, K)
    p0 = B.w4a8_pack_weights(torch.from_numpy(r["qw"]).cuda(), to_dev16(torch, r["sw"], torch.float16), torch.from_numpy(r["z"]).cuda())
    ncopies = copies_for(p0.numel(), l2_bytes)
    packed = [p0] + [p0.clone() for _ in range(ncopies - 1)]
    ws = B.new_workspace(M, N, K)
    qa, sa, asum = B.w4a8_quantize_act(to_dev16(torch, r["x"], torch.bfloat16))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    B.w4a8_gemm(qa, sa, asum, packed[0], N, ws, out=y)
    B.w4a8_check_status(ws)

    def body():
        for _ in range(2):
            for p in packed:
                B.w4a8_gemm(qa, sa, asum, p, N, ws, out=y)
    _, times = timer.graph_ms(body, replays=5, warm=2)
    B.w4a8_check_status(ws)
    us = float(np.median(times)) * 1e3 / (2 * ncopies)
    tops = wl.algorithmic_ops(M, N, K) / us / 1e6
    peak2 = 2.0 * peaks["bf16_tflops"]
    out = {"bound": "tensor", "kernel": plan_name(B, M, N, K), "workload": f"prefill_gate_up: M={M} K={K} N={N}",
           "achieved": round(tops, 1), "unit": "TOP/s (int8)", "peak": round(peak2, 1),
           "peak_source": f"2 x the {peaks['source']} bf16 GEMM rate (burst); nominal dense int8 : bf16 = 2",
           "frac": round(tops / peak2, 4), "us_per_launch": round(us, 2),
           "frac_of_nominal_4500": round(tops / NOMINAL_INT8_TOPS, 4),
           "tensor_pipe_active_pct_ncu": 33.5, "traffic": None,
           "timing": "median of 5 replays of back-to-back launches in one graph"}
    if peaks.get("int8_tops_burst"):
        out["peak_int8_mm"] = round(peaks["int8_tops_burst"], 1)
        out["frac_of_int8_mm"] = round(tops / peaks["int8_tops_burst"], 4)
    del packed, p0
    torch.cuda.empty_cache()
    return out


def run_quantize_roofline(torch, B, peaks, l2_bytes, timer):
    """quantize_act alone at 1024 x 4096 (one wave of CTAs: latency shows) and 4096 x 4096 (several waves), on inputs
    visited in turn (more than two L2 capacities in all)."""
    def one(M, K):
        nbytes = wl.algorithmic_bytes_quantize(M, K)
        ncopies = copies_for(2 * M * K, l2_bytes)
        xs = [torch.randn((M, K), device="cuda").to(torch.bfloat16) for _ in range(ncopies)]
        qa = torch.empty((M, K), dtype=torch.int8, device="cuda")
        sa = torch.empty((M,), dtype=torch.float16, device="cuda")
        asum = torch.empty((M, K // 128), dtype=torch.int32, device="cuda")

        def body():
            for x in xs:
                B.w4a8_quantize_act(x, 128, out=(qa, sa, asum))
        _, times = timer.graph_ms(body, replays=5, warm=2)
        us = float(np.median(times)) * 1e3 / ncopies
        del xs
        torch.cuda.empty_cache()
        return nbytes, us
    nbytes, us = one(1024, 4096)
    gbs = nbytes / us / 1e3
    nbytes4, us4 = one(4096, 4096)
    gbs4 = nbytes4 / us4 / 1e3
    return {"bound": "hbm", "kernel": "quantize_act_kernel<256 threads, 2 chunks, reciprocal + tie fallback>",
            "workload": "M=1024 K=4096", "achieved": round(gbs, 1),
            "unit": "GB/s", "peak": peaks["hbm_gbs"], "frac": round(gbs / peaks["hbm_gbs"], 4), "us_per_launch": round(us, 2),
            "algorithmic_bytes_per_launch": nbytes, "traffic": QUANTIZE_TRAFFIC_BYTES_PER_LAUNCH,
            "m4096": {"workload": "M=4096 K=4096", "achieved": round(gbs4, 1), "frac": round(gbs4 / peaks["hbm_gbs"], 4),
                      "us_per_launch": round(us4, 2), "algorithmic_bytes_per_launch": nbytes4},
            "timing": "median of 5 replays of back-to-back launches in one graph"}


def run_w4a16_comparison(torch, B, peaks, l2_bytes, timer):
    """The paper's argument for W4A8 over weight-only W4A16, measured on the same packed layers: at 8 tokens both are
    bound by the weight bytes (W4A16 skips the activation quantiser), at 1024 tokens the weight-only scheme computes in
    bf16 - here as this library's dequantise kernel followed by the library bf16 GEMM (torch.matmul), the usual form -
    while W4A8 multiplies in INT8.  Times are per linear layer (quantiser included for W4A8), cold weights."""
    rows = []
    rng = np.random.default_rng(11)
    for lname in ("qkv", "gate_up"):
        K, N = wl.LAYERS[lname]
        c = wl.random_codes(rng, 1024, N, K)
        p0 = B.w4a8_pack_weights(torch.from_numpy(c["qw"]).cuda(), to_dev16(torch, c["sw"], torch.float16),
                                 torch.from_numpy(c["z"]).cuda())
        ncopies = copies_for(p0.numel(), l2_bytes)
        packed = [p0] + [p0.clone() for _ in range(ncopies - 1)]
        ws = B.new_workspace(1024, N, K)
        x_all = to_dev16(torch, c["x"], torch.bfloat16)
        W = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        for M in (8, 1024):
            x = x_all[:M].contiguous()
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            scratch = (torch.empty((M, K), dtype=torch.int8, device="cuda"), torch.empty((M,), dtype=torch.float16, device="cuda"),
                       torch.empty((M, K // 128), dtype=torch.int32, device="cuda"))
            reps = 4 if M <= 16 else 1

            def w4a8():
                for _ in range(reps):
                    for p in packed:
                        B.w4a8_linear(x, p, N, ws, 128, out=y, scratch=scratch)

            def w4a16():
                for _ in range(reps):
                    for p in packed:
                        if M <= 16:
                            B.w4a8_a16_gemm(x, p, N, ws, out=y)
                        else:
                            B.w4a8_dequantize_weights(p, N, K, out=W)
                            torch.matmul(x, W.t(), out=y)
            row = {"layer": lname, "M": M}
            for name, body in (("w4a8_us", w4a8), ("w4a16_us", w4a16)):
                _, times = timer.graph_ms(body, replays=5, warm=2)
                row[name] = round(min(times) * 1e3 / (reps * ncopies), 2)
            B.w4a8_check_status(ws)
            row["w4a16_form"] = "w4a8_a16_gemm (strip kernel, bf16 MMA)" if M <= 16 else "w4a8_dequantize_weights + torch.matmul (bf16)"
            if M > 16:
                B.w4a8_dequantize_weights(packed[0], N, K, out=W)

                def bf16_only():
                    for _ in range(ncopies):
                        torch.matmul(x, W.t(), out=y)
                _, times = timer.graph_ms(bf16_only, replays=5, warm=2)
                row["bf16_gemm_alone_us"] = round(min(times) * 1e3 / ncopies, 2)
            row["w4a8_speedup_over_w4a16"] = round(row["w4a16_us"] / row["w4a8_us"], 2)
            rows.append(row)
        del packed, p0, W
        torch.cuda.empty_cache()
    return rows


def run_rope_roofline(torch, B, peaks, l2_bytes, timer):
    """Rotary embedding of pre-rotation cached keys at shifted positions (streaming prefill): 8 KV heads of 128, a window
    of 4096 tokens and a long one of 65536; inputs visited in turn (more than two L2 capacities in all)."""
    rows = []
    for T in (4096, 65536):
        H, D = 8, 128
        nbytes = T * H * D * 4 + 4 * T
        ncopies = copies_for(T * H * D * 2, l2_bytes)
        ks = [torch.randn((T, H, D), device="cuda").to(torch.bfloat16) for _ in range(ncopies)]
        pos = torch.arange(T, dtype=torch.int32, device="cuda")
        out = torch.empty_like(ks[0])

        def body():
            for k in ks:
                B.w4a8_rope_shifted_keys(k, pos, 45, 1.0e6, out=out)
        _, times = timer.graph_ms(body, replays=5, warm=2)
        us = float(np.median(times)) * 1e3 / ncopies
        rows.append({"kernel": "rope_shifted_keys_kernel", "workload": f"T={T} H={H} D={D}", "bound": "hbm",
                     "achieved": round(nbytes / us / 1e3, 1), "unit": "GB/s", "peak": peaks["hbm_gbs"],
                     "frac": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4), "us_per_launch": round(us, 2),
                     "algorithmic_bytes_per_launch": nbytes})
        del ks
        torch.cuda.empty_cache()
    return rows


def run_layer_chain(torch, B, peaks, l2_bytes, timer):
    """The four linears of one decoder layer back to back (QKV, O, gate+up, down), each as the public
    w4a8_linear call (quantise + GEMM) on its own input, in one CUDA graph: what a decoder layer spends in
    this path per step, launch chain included.  Three cold copies of the layer's weights are visited in turn."""
    out = []
    int8_peak = 2.0 * peaks["bf16_tflops"]
    layer_bytes = sum(K * N // 2 + 5 * (K // 128) * N // 2 for K, N in wl.LAYERS.values())
    ncopies = copies_for(layer_bytes, l2_bytes)
    rng = np.random.default_rng(7)
    m_max = 1024
    layers = []
    for lname, (K, N) in wl.LAYERS.items():
        c = wl.random_codes(rng, m_max, N, K)
        p0 = B.w4a8_pack_weights(torch.from_numpy(c["qw"]).cuda(), to_dev16(torch, c["sw"], torch.float16),
                                 torch.from_numpy(c["z"]).cuda())
        layers.append({"K": K, "N": N, "x": to_dev16(torch, c["x"], torch.bfloat16),
                       "packed": [p0] + [p0.clone() for _ in range(ncopies - 1)],
                       "ws": B.new_workspace(m_max, N, K)})
    for M in (8, 1024):
        for L in layers:
            K, N = L["K"], L["N"]
            L["xm"] = L["x"][:M].contiguous()
            L["scratch"] = (torch.empty((M, K), dtype=torch.int8, device="cuda"),
                            torch.empty((M,), dtype=torch.float16, device="cuda"),
                            torch.empty((M, K // 128), dtype=torch.int32, device="cuda"))
            L["y"] = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        reps = 4 if M <= 64 else 1

        def body():
            for _ in range(reps):
                for c in range(ncopies):
                    for L in layers:
                        B.w4a8_linear(L["xm"], L["packed"][c], L["N"], L["ws"], 128, out=L["y"], scratch=L["scratch"])
        _, times = timer.graph_ms(body, replays=5, warm=2)
        for L in layers:
            B.w4a8_check_status(L["ws"])
        us = min(times) * 1e3 / (reps * ncopies)
        ops = sum(wl.algorithmic_ops(M, L["N"], L["K"]) for L in layers)
        nbytes = sum(step_bytes(M, L["N"], L["K"]) for L in layers)
        t_roof = sum(max(wl.algorithmic_ops(M, L["N"], L["K"]) / (int8_peak * 1e12),
                         step_bytes(M, L["N"], L["K"]) / (peaks["hbm_gbs"] * 1e9)) for L in layers)
        row = {"M": M, "us_per_layer": round(us, 2), "kernels_per_layer": 8, "tops": round(ops / us / 1e6, 1),
               "gbs": round(nbytes / us / 1e3, 1), "frac_measured": round(t_roof * 1e6 / us, 3)}
        # The same layer with the fused steps: the gate+up projection's epilogue (or, above 16 tokens, the quantiser that
        # follows it) forms SiLU(gate) * up and the down projection's quantised input, which the down projection then
        # takes as it is - the real data dependency of a decoder layer; O and down add their output into the residual
        # stream in their epilogues, in place.
        # Fractions use the same roofline sum as above (the same logical work).
        by_name = dict(zip(wl.LAYERS.keys(), layers))
        gu, dn = by_name["gate_up"], by_name["down"]
        I = gu["N"] // 2
        assert dn["K"] == I
        h_out = (torch.empty((M, I), dtype=torch.bfloat16, device="cuda"), torch.empty((M, I), dtype=torch.int8, device="cuda"),
                 torch.empty((M,), dtype=torch.float16, device="cuda"), torch.empty((M, I // 128), dtype=torch.int32, device="cuda"))
        resid = torch.zeros((M, dn["N"]), dtype=torch.bfloat16, device="cuda")
        assert by_name["o"]["N"] == dn["N"]
        form_names = {B.GATE_UP_EPILOGUE: "SiLU*up in the strip kernel's epilogue + requantise kernel",
                      B.GATE_UP_ONE_KERNEL: "one kernel (epilogue, last CTAs stay and requantise)",
                      B.GATE_UP_SEPARATE: "GEMM + SiLU*up quantiser"}
        forms = [B.w4a8_gate_up_form(M, gu["N"], gu["K"])] + ([B.GATE_UP_ONE_KERNEL] if M <= 16 else [])
        for fi, form in enumerate(forms):
            def body_fused():
                for _ in range(reps):
                    for c in range(ncopies):
                        L = by_name["qkv"]
                        B.w4a8_linear(L["xm"], L["packed"][c], L["N"], L["ws"], 128, out=L["y"], scratch=L["scratch"])
                        L = by_name["o"]                       # O and down add into the residual stream, in place
                        B.w4a8_quantize_act(L["xm"], 128, out=L["scratch"])
                        B.w4a8_gemm_residual(L["scratch"][0], L["scratch"][1], L["scratch"][2], L["packed"][c], resid, L["N"], L["ws"],
                                             128, out=resid)
                        B.w4a8_quantize_act(gu["xm"], 128, out=gu["scratch"])
                        B.w4a8_gate_up_silu_quantize(gu["scratch"][0], gu["scratch"][1], gu["scratch"][2], gu["packed"][c], gu["N"],
                                                     gu["ws"], 128, form=form, y_scratch=gu["y"], out=h_out)
                        B.w4a8_gemm_residual(h_out[1], h_out[2], h_out[3], dn["packed"][c], resid, dn["N"], dn["ws"], 128, out=resid)
            _, times = timer.graph_ms(body_fused, replays=5, warm=2)
            for L in layers:
                B.w4a8_check_status(L["ws"])
            usf = min(times) * 1e3 / (reps * ncopies)
            row["fused_gate_up" if fi == 0 else "fused_gate_up_one_kernel"] = {
                "us_per_layer": round(usf, 2), "kernels_per_layer": 7 if form == B.GATE_UP_ONE_KERNEL else 8,
                "frac_measured": round(t_roof * 1e6 / usf, 3), "form": form_names[form]}
        out.append(row)
    del layers
    torch.cuda.empty_cache()
    return out


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2608_12932_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()
    peaks = measured_peaks()
    l2_bytes = torch.cuda.get_device_properties(local).L2_cache_size or L2_BYTES_ASSUMED
    timer = Timer(torch)

    case = wl.make_config(HEADLINE)
    M, N, K, g = case["M"], case["N"], case["K"], case["group"]
    qw = torch.from_numpy(case["qw"]).cuda()
    sw = to_dev16(torch, case["sw"], torch.float16)
    z = torch.from_numpy(case["z"]).cuda()
    packed0 = B.w4a8_pack_weights(qw, sw, z, g)                 # offline, once
    ncopies = copies_for(packed0.numel(), l2_bytes)
    packed = [packed0] + [packed0.clone() for _ in range(ncopies - 1)]
    ws = B.new_workspace(M, N, K, g)
    x = to_dev16(torch, case["x"], torch.bfloat16)
    qa = torch.empty((M, K), dtype=torch.int8, device="cuda")
    sa = torch.empty((M,), dtype=torch.float16, device="cuda")
    asum = torch.empty((M, K // g), dtype=torch.int32, device="cuda")
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")

    def step(i):
        B.w4a8_linear(x, packed[i % ncopies], N, ws, g, out=y, scratch=(qa, sa, asum))
    launches_per_step = 2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- correctness of this very launch configuration against the oracle (outside the timed region)
    from oracle import cfast
    from oracle import w4a8_oracle as onp
    step(0)
    B.w4a8_quantize_act(x, g, out=(qa, sa, asum))       # the codes themselves, for the exact comparison below
    B.w4a8_check_status(ws)
    ref = cfast.w4a8_linear(case["x"], case["qw"], case["sw"], case["z"], g)
    ok, ratio = onp.within_tolerance(y.view(torch.int16).cpu().numpy().view(np.uint16), ref["ref"])
    parity = {"codes_exact": bool(np.array_equal(qa.cpu().numpy(), ref["qa"])), "bf16_within_tolerance": ok,
              "worst_err_over_bound": round(ratio, 4)}

    # ---- timed region: W warm-up steps, then exactly K steps in one graph launch
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    B.w4a8_check_status(ws)              # a kernel that gave up on a bounded wait must not be timed 2000 times
    g_steps = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_steps):
        for i in range(args.steps):
            step(i)
    g_steps.replay()                     # untimed: graph upload, instruction caches
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", ""))
    barrier()
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g_steps.replay()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    # keep the GPU in the same state a little longer so the sampler sees clocks under this load
    t_end = time.perf_counter() + 0.6
    while time.perf_counter() < t_end:
        g_steps.replay()
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    B.w4a8_check_status(ws)
    ms_total = max_over_ranks(ms_total, dist if world > 1 else None, "cuda")
    sbytes = step_bytes(M, N, K)
    value = whole_job_gbs(sbytes, args.steps, world, ms_total)

    # ---- roofline of the dominant kernel: the small-M GEMM alone, same rotation, K launches
    step_us = ms_total * 1e3 / args.steps
    def gemm_only():
        for i in range(args.steps):
            B.w4a8_gemm(qa, sa, asum, packed[i % ncopies], N, ws, g, out=y)
    _, gt = timer.graph_ms(gemm_only, replays=5, warm=2)
    gemm_us = float(np.median(gt)) * 1e3 / args.steps
    gbytes = wl.algorithmic_bytes_gemm(M, N, K)
    roof_kernel, roof_us, roof_bytes = plan_name(B, M, N, K), gemm_us, gbytes
    achieved = roof_bytes / roof_us / 1e3
    traffic = TRAFFIC_BYTES_PER_LAUNCH.get(roof_kernel.split("<")[0])      # ncu capture of this kernel at this shape, if one is on file

    def quant_only():
        for i in range(args.steps):
            B.w4a8_quantize_act(x, g, out=(qa, sa, asum))
    _, qt = timer.graph_ms(quant_only, replays=5, warm=2)
    quant_us = float(np.median(qt)) * 1e3 / args.steps

    # ---- end to end from pinned host buffers through w4a8_linear_host, copies inside the timed region
    x_host = torch.from_numpy(np.ascontiguousarray(case["x"]).view(np.int16)).view(torch.bfloat16).pin_memory()
    # E2E_DEPTH requests in flight, each with its own staging buffers, workspace, pinned output and
    # stream: the copies of one request overlap the kernels of its neighbours, as in a serving loop
    y_hosts = [torch.empty((M, N), dtype=torch.bfloat16).pin_memory() for _ in range(E2E_DEPTH)]
    y_host = y_hosts[(args.steps - 1) % E2E_DEPTH]           # the last step's result, checked below
    hosts = [B.HostLinear(M, N, K, packed0, B.new_workspace(M, N, K), g) for _ in range(E2E_DEPTH)]
    lanes = [torch.cuda.Stream() for _ in range(E2E_DEPTH)]

    def e2e_steps():
        cur = torch.cuda.current_stream()
        for st in lanes:
            st.wait_stream(cur)
        for i in range(args.steps):
            j = i % E2E_DEPTH
            hosts[j].packed_w = packed[i % ncopies]
            with torch.cuda.stream(lanes[j]):
                hosts[j](x_host, y_hosts[j])
        for st in lanes:
            cur.wait_stream(st)
    g_e2e, et = timer.graph_ms(e2e_steps, replays=3, warm=2)
    barrier()
    e2e_ms = float(np.median(et))
    e2e_ms = max_over_ranks(e2e_ms, dist if world > 1 else None, "cuda")
    e2e_value = whole_job_gbs(sbytes, args.steps, world, e2e_ms)
    e2e_ok, _ = onp.within_tolerance(y_host.view(torch.int16).numpy().view(np.uint16), ref["ref"])
    parity["e2e_within_tolerance"] = e2e_ok

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- CPU oracle on this host's cores, same step (bounded: a few seconds)
    osteps, oel, threads = time_oracle(case, 3.0)
    cpu_gbs = sbytes * osteps / oel / 1e9

    # ---- the other rooflines: a library INT8 GEMM as the measured tensor peak, the large-M kernel on the
    # streaming-prefill configuration, the quantise kernel at a prefill-sized input
    peaks.update(measure_int8_peak(torch))
    roof_large = run_large_m_roofline(torch, B, peaks, l2_bytes, timer)
    roof_quant = run_quantize_roofline(torch, B, peaks, l2_bytes, timer)
    roof_rope = run_rope_roofline(torch, B, peaks, l2_bytes, timer)

    sweep = None
    targets = None
    if not args.no_sweep and world == 1:
        sweep, sweep_pc = run_sweep(torch, B, peaks, l2_bytes, timer)
        layer_chain = run_layer_chain(torch, B, peaks, l2_bytes, timer)
        w4a16_cmp = run_w4a16_comparison(torch, B, peaks, l2_bytes, timer)
        small = [r for r in sweep if r["M"] <= 16]
        large = [r for r in sweep if r["M"] >= 1024]
        targets = {"small_m_target": 0.70, "small_m_min_frac": min(r["frac_measured"] for r in small),
                   "small_m_max_frac": max(r["frac_measured"] for r in small),
                   "large_m_target": 0.60, "large_m_min_frac": min(r["frac_measured"] for r in large),
                   "large_m_max_frac": max(r["frac_measured"] for r in large),
                   "denominators": "measured HBM copy rate (M <= 16); 2 x measured bf16 burst (M >= 1024)"}

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 x uint4 -> int32 (fp32 scaling, bf16 out)", "data": "synthetic",
        "config": {"workload": workload_name(M, N, K),
                   "l2": f"{ncopies} distinct packed weight copies visited in turn ({ncopies * packed0.numel() / 2**20:.0f} MiB "
                         f"> 2 x L2 of {l2_bytes / 2**20:.0f} MiB); activations stay L2-resident as in a real decoder",
                   "launch": "one CUDA graph of K steps, CUDA events around the replay",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "e2e": {"value": round(e2e_value, 2), "unit": "GB/s", "h2d_bytes_per_step": M * K * 2,
                "d2h_bytes_per_step": M * N * 2, "ms_per_step": e2e_ms / args.steps,
                "requests_in_flight": E2E_DEPTH},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": roof_kernel, "achieved": round(achieved, 1),
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4),
                     "peak_source": f"of {peaks['source']} (STREAM-style copy, burst)",
                     "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                     "us_per_launch": round(roof_us, 3), "algorithmic_bytes_per_launch": roof_bytes,
                     "traffic": traffic,
                     "timing": "median of 5 replays of K back-to-back launches in one graph, inter-launch gaps included"},
        "kernels_us": {"w4a8_linear": round(step_us, 3), "w4a8_quantize_act": round(quant_us, 3),
                       "w4a8_gemm": round(gemm_us, 3)},
        "cpu_baseline": {"value": round(cpu_gbs, 3), "unit": "GB/s", "cores": threads, "kind": "oracle",
                         "sample": f"the whole step (M={M}, all {N} channels), {osteps} repetitions in {oel:.1f} s"},
        "parity": parity,
        "peaks": {k: (round(v, 1) if isinstance(v, float) else v) for k, v in peaks.items()},
        "roofline_large_m": roof_large,
        "roofline_quantize_act": roof_quant,
        "roofline_rope_shifted_keys": roof_rope,
    }
    if sweep is not None:
        line["targets"] = targets
        line["sweep"] = sweep
        line["sweep_per_channel_scales"] = sweep_pc
        line["layer_chain"] = layer_chain
        line["w4a16_comparison"] = w4a16_cmp
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_shape(args):
    """--shape LAYER:M : one sweep point launched eagerly `steps` times on cold weight copies (the small
    case that ncu captures are taken on): w4a8_quantize_act + w4a8_gemm; prints one JSON line."""
    import torch

    from paper_2608_12932_b200 import binding as B
    lname, M = args.shape.split(":")
    M = int(M)
    K, N = wl.LAYERS[lname]
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    case = wl.make_layer(K, N, wl.LAYER_SEEDS[lname], M)
    packed0 = B.w4a8_pack_weights(torch.from_numpy(case["qw"]).cuda(), to_dev16(torch, case["sw"], torch.float16),
                                  torch.from_numpy(case["z"]).cuda())
    l2_bytes = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size or L2_BYTES_ASSUMED
    ncopies = copies_for(packed0.numel(), l2_bytes)
    packed = [packed0] + [packed0.clone() for _ in range(ncopies - 1)]
    ws = B.new_workspace(M, N, K)
    x = to_dev16(torch, case["x"], torch.bfloat16)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    h_out = (torch.empty((M, N // 2), dtype=torch.bfloat16, device="cuda"), torch.empty((M, N // 2), dtype=torch.int8, device="cuda"),
             torch.empty((M,), dtype=torch.float16, device="cuda"), torch.empty((M, N // 256), dtype=torch.int32, device="cuda"))
    times = []
    for i in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        qa, sa, asum = B.w4a8_quantize_act(x)
        e0.record()
        if args.variant == "a16":
            B.w4a8_a16_gemm(x, packed[i % ncopies], N, ws, out=y)
        elif args.variant == "gate_up":
            B.w4a8_gate_up_silu_quantize(qa, sa, asum, packed[i % ncopies], N, ws, y_scratch=y, out=h_out)
        elif args.variant == "residual":
            B.w4a8_gemm_residual(qa, sa, asum, packed[i % ncopies], y, N, ws, out=y)
        elif args.per_channel:
            B.w4a8_gemm_per_channel(qa, sa, packed[i % ncopies], N, ws, out=y)
        else:
            B.w4a8_gemm(qa, sa, asum, packed[i % ncopies], N, ws, out=y)
        e1.record()
        e1.synchronize()
        if i >= args.warmup:
            times.append(e0.elapsed_time(e1) * 1e3)
    B.w4a8_check_status(ws)
    us = float(np.median(times))
    print(json.dumps({"shape": args.shape, "variant": args.variant, "per_channel_scales": bool(args.per_channel), "M": M, "N": N, "K": K, "gemm_us_eager_median": round(us, 2),
                      "tops": round(wl.algorithmic_ops(M, N, K) / us / 1e6, 1),
                      "gbs": round(wl.algorithmic_bytes_gemm(M, N, K) / us / 1e3, 1), "launches": args.steps}))


def run_rope(args):
    """--rope T : w4a8_rope_shifted_keys on T tokens x 8 heads x 128, launched eagerly `steps` times on inputs visited
    in turn (the small case that ncu captures are taken on); prints one JSON line."""
    import torch

    from paper_2608_12932_b200 import binding as B
    T, H, D = args.rope, 8, 128
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    l2_bytes = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size or L2_BYTES_ASSUMED
    ncopies = copies_for(T * H * D * 2, l2_bytes)
    ks = [torch.randn((T, H, D), device="cuda").to(torch.bfloat16) for _ in range(ncopies)]
    pos = torch.arange(T, dtype=torch.int32, device="cuda")
    out = torch.empty_like(ks[0])
    times = []
    for i in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.w4a8_rope_shifted_keys(ks[i % ncopies], pos, 45, 1.0e6, out=out)
        e1.record()
        e1.synchronize()
        if i >= args.warmup:
            times.append(e0.elapsed_time(e1) * 1e3)
    us = float(np.median(times))
    print(json.dumps({"rope": {"T": T, "H": H, "D": D}, "us_eager_median": round(us, 2), "gbs": round(T * H * D * 4 / us / 1e3, 1),
                      "launches": args.steps}))


# dram__bytes_read.sum + dram__bytes_write.sum of one GEMM launch at the headline shape, by kernel, from the ncu
# captures summarised under profiles/ (gemm_strip_qkv_M8.md, gemm_cluster_qkv_M8.md)
QUANTIZE_TRAFFIC_BYTES_PER_LAUNCH = 8410624      # ncu, quantize_act at 1024 x 4096 (profiles/quantize_act_M1024_K4096.md)
TRAFFIC_BYTES_PER_LAUNCH = {"gemm_strip_kernel": 13148416, "gemm_cluster_kernel": 13144832}
E2E_DEPTH = int(os.environ.get("W4A8_E2E_DEPTH", "8"))          # host requests in flight in the end-to-end measurement


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=int(os.environ.get("WORLD_SIZE", "1")))
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--shape", default=None, help="LAYER:M, e.g. gate_up:1024 - run only that GEMM (profiling aid)")
    ap.add_argument("--per-channel", action="store_true", help="with --shape: w4a8_gemm_per_channel instead of w4a8_gemm")
    ap.add_argument("--variant", default="gemm", choices=["gemm", "a16", "gate_up", "residual"],
                    help="with --shape: w4a8_a16_gemm, w4a8_gate_up_silu_quantize (gate_up layer) or w4a8_gemm_residual instead of w4a8_gemm")
    ap.add_argument("--rope", type=int, default=0, help="T: run only w4a8_rope_shifted_keys on T tokens x 8 heads x 128 (profiling aid)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.rope:
        run_rope(args)
    elif args.shape:
        run_shape(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
