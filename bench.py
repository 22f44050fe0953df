#!/usr/bin/env python
"""Benchmark of the per-example-statistics hot path on B200.

One step = one pass of the whole path over one batch of a bf16 linear layer.  The default workload is the
large layer (B=256, T=1024, d_in=2048, d_out=8192; X ~ N(0,1), dY Student-t(3)/sqrt(T)); `--workload c2` is
the transformer-MLP-shaped layer (B=64, T=256, d_in=512, d_out=2048, 10% of sequences x5):
  pe_linear_stats_all      -> sum_b G_b, sum_b G_b^2 and sum_b sign(G_b) in one pass   (tcgen05 kernel)
  per-token statistic      -> sum_{b,t} dY^2 X^2   (pe_token_sqstats: squares on chip, tf32 tcgen05 kernel;
                              from 1e8 input elements on pe_token_sqstats_staged: half squares, 16-bit rate)
  microadam_step           on fp32 master weights (+ bf16 copy)
  microsignsgd_step        on a second set of master weights (+ bf16 copy)
`value` is the contraction throughput of the whole step: 2 x (2*B*T*d_in*d_out) flops (the per-example and the
per-token contraction) over the step time.  The headline `roofline` entry is the per-example statistics kernel
of the step; `pe_linear_stats` holds the call the target is stated on (phi = square, both outputs) timed in
the same run, interleaved call by call with the cuBLAS batch weight-gradient GEMM of the same shape.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c4] [--impl ours|reference]
  python bench.py --sweep          (single-layer shape sweep, one JSON line per point)

With N > 1 (torchrun) every rank runs an independent replica of the same workload on its own GPU
(the path has no exchange step); the reported value is the sum over ranks divided by the slowest
rank's time.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "per-example-stat TFLOP/s"
UNIT = "TFLOP/s"
WORKLOADS = {
    # name: (B, T, d_in, d_out, rotating input sets)
    "c2": (64, 256, 512, 2048, 6),
    "c4": (256, 1024, 2048, 8192, 1),
    "c4s": (16, 1024, 2048, 8192, 1),     # a 16-sequence slice of c4 (335 MB of inputs): small enough to profile
}
TOKEN_STAGED_MIN_ELEMS = 100_000_000
ADAM = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)
SIGN = dict(lr=3.47e-3, beta=0.9)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def profile_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of one kernel from the committed ncu summaries, if present (a line
    "dram_bytes_per_launch <kernel>: <bytes>").  The large layer's figures (lines "dram_bytes_per_launch_c4 ...")
    come from a capture of full-size launches with the two DRAM byte counters alone, which take a single pass."""
    fname, tag = {"c2": ("c2", "dram_bytes_per_launch"), "c4s": ("c4_slice", "dram_bytes_per_launch"),
                  "c4": ("c4_slice", "dram_bytes_per_launch_c4")}.get(workload, (workload, "dram_bytes_per_launch"))
    path = os.path.join(ROOT, "profiles", f"tc_stats_kernel_{fname}.txt")
    key = f"{tag} {kernel}:"
    try:
        for line in open(path):
            if line.startswith(key):
                return float(line[len(key):].split()[0])
    except OSError:
        pass
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100", "-i", str(self.gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx = float(parts[2])
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(torch, dist, ms: float, device) -> float:
    """Slowest rank's time (every rank gets the same answer); identity without a process group."""
    if dist is None:
        return float(ms)
    tt = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def replica_throughput(world: int, flops_per_step: float, ms_per_step: float) -> float:
    """Whole-job TFLOP/s of `world` independent replicas that all take the slowest rank's step time."""
    return world * flops_per_step / (ms_per_step * 1e-3) / 1e12


def make_state(pe, inputs, torch, name, dev, seed_offset=0):
    B, T, d_in, d_out, nsets = WORKLOADS[name]
    sets = []
    for k in range(nsets):
        if name == "c2":
            li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=inputs.BASE_SEED + 2 + 1000 * k + seed_offset, device=dev,
                                            name="c2", with_weights=(k == 0))
        else:
            li = inputs.heavy_tailed_layer(B, T, d_in, d_out, seed=inputs.BASE_SEED + 4 + 1000 * k + seed_offset, device=dev,
                                           name=name, with_weights=(k == 0))
        sets.append(li)
    n = d_out * d_in
    f32 = dict(dtype=torch.float32, device=dev)
    st = {
        "shape": (B, T, d_in, d_out), "sets": sets,
        "mean": torch.empty((d_out, d_in), **f32), "sq": torch.empty((d_out, d_in), **f32),
        "sgn": torch.empty((d_out, d_in), **f32), "tok": torch.empty((d_out, d_in), **f32),
        "theta": sets[0].W.clone(), "m": torch.zeros((d_out, d_in), **f32), "v": torch.zeros((d_out, d_in), **f32),
        "theta_lp": torch.empty((d_out, d_in), dtype=torch.bfloat16, device=dev),
        "theta2": sets[0].W.clone(), "m2": torch.zeros((d_out, d_in), **f32),
        "theta2_lp": torch.empty((d_out, d_in), dtype=torch.bfloat16, device=dev),
        "n": n,
    }
    # Per-token statistic: the one-kernel tf32 form on small layers; from about 1e8 input elements on, the
    # two-pass form (half operands at the full 16-bit tensor rate) with a caller-owned workspace.
    st["tok_ws"] = None
    if B * T * (d_in + d_out) >= TOKEN_STAGED_MIN_ELEMS:
        need = pe.pe_token_sqstats_staged_workspace_bytes(B, T, d_in, d_out)
        if need > 0:
            st["tok_ws"] = torch.empty(need, dtype=torch.uint8, device=dev)
    return st


def token_stat(pe, st, X, dY):
    if st["tok_ws"] is not None:
        pe.pe_token_sqstats_staged(X, dY, st["tok"], st["tok_ws"])
    else:
        pe.pe_token_sqstats(X, dY, st["tok"])


def run_step(pe, st, i, X=None, dY=None, ev=None):
    B = st["shape"][0]
    li = st["sets"][i % len(st["sets"])]
    X = li.X if X is None else X
    dY = li.dY if dY is None else dY
    if ev is not None:
        ev[0].record()
    pe.pe_linear_stats_all(X, dY, st["mean"], st["sq"], st["sgn"])      # sum G_b, sum G_b^2 and sum sign(G_b) in one pass
    if ev is not None:
        ev[1].record()
    token_stat(pe, st, X, dY)
    if ev is not None:
        ev[2].record()
    pe.microadam_step(st["theta"], st["m"], st["v"], st["mean"], st["sq"], B, step=i + 1, theta_lp=st["theta_lp"], **ADAM)
    pe.microsignsgd_step(st["theta2"], st["m2"], st["sgn"], B, theta_lp=st["theta2_lp"], **SIGN)


def time_region(torch, fn, iters):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(iters):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters


def time_each(torch, fn, iters=20, warmup=3):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    ts = []
    for i in range(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(i); b.record()
        ts.append((a, b))
    torch.cuda.synchronize()
    v = sorted(x.elapsed_time(y) for x, y in ts)
    return v[len(v) // 2], v[0]


def time_interleaved(torch, fns, iters=20, warmup=3):
    """Times several calls in alternation (a, b, a, b, ...), each call between its own pair of events, so
    that all of them see the same clocks and thermal state.  Returns [(median_ms, best_ms)] per call."""
    for i in range(warmup):
        for fn in fns:
            fn(i)
    torch.cuda.synchronize()
    evs = [[] for _ in fns]
    for i in range(iters):
        for k, fn in enumerate(fns):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(i); b.record()
            evs[k].append((a, b))
    torch.cuda.synchronize()
    out = []
    for e in evs:
        v = sorted(x.elapsed_time(y) for x, y in e)
        out.append((v[len(v) // 2], v[0]))
    return out


def target_call_numbers(torch, pe, st, li, peaks):
    """The call the throughput target is stated on: pe_linear_stats(phi = square) with both outputs, timed
    call by call in alternation with the cuBLAS batch weight-gradient GEMM of the same shape."""
    B, T, d_in, d_out = st["shape"]
    flops_one = 2.0 * B * T * d_in * d_out
    A2, B2 = li.dY.view(B * T, d_out), li.X.view(B * T, d_in)
    (med, best), (med_g, best_g) = time_interleaved(
        torch, [lambda i: pe.pe_linear_stats(li.X, li.dY, pe.PHI_SQUARE, st["mean"], st["sq"]),
                lambda i: torch.matmul(A2.t(), B2)])
    tf = flops_one / med / 1e9
    return {"call": "pe_linear_stats(phi=square, out_mean + out_stat)", "ms_median": med, "ms_best": best, "tflops": tf,
            "frac_of_peak_burst": tf / peaks["bf16_tflops"], "frac_of_peak_sustained": tf / peaks["bf16_tflops_sustained"],
            "peak_source": peaks["source"], "gemm": "torch.matmul(dY_flat^T, X_flat), bf16 (cuBLAS)",
            "gemm_ms_median": med_g, "gemm_ms_best": best_g, "gemm_tflops": flops_one / med_g / 1e9,
            "overhead_vs_gemm": med / med_g, "overhead_vs_gemm_best": best / best_g,
            "timing": "20 calls each, alternating, one CUDA-event pair per call, after 3 warm-ups"}


def context_numbers(torch, pe, st, li, peaks, dev):
    """Per-kernel timings taken alone, outside the timed region: each statistics call, the cuBLAS batch
    weight-gradient GEMM of the same shape, and the update kernels on a parameter count far beyond L2."""
    B, T, d_in, d_out = st["shape"]
    flops_one = 2.0 * B * T * d_in * d_out
    extra = {}
    med, best = time_each(torch, lambda i: pe.pe_linear_stats(li.X, li.dY, pe.PHI_SQUARE, st["mean"], st["sq"]))
    extra["pe_linear_stats_square_us"] = {"median": med * 1e3, "best": best * 1e3, "tflops_median": flops_one / med / 1e9}
    med_s, best_s = time_each(torch, lambda i: pe.pe_linear_stats(li.X, li.dY, pe.PHI_SIGN, None, st["sgn"]))
    extra["pe_linear_stats_sign_us"] = {"median": med_s * 1e3, "best": best_s * 1e3, "tflops_median": flops_one / med_s / 1e9}
    med_a3, best_a3 = time_each(torch, lambda i: pe.pe_linear_stats_all(li.X, li.dY, st["mean"], st["sq"], st["sgn"]))
    extra["pe_linear_stats_all_us"] = {"median": med_a3 * 1e3, "best": best_a3 * 1e3, "tflops_median": flops_one / med_a3 / 1e9}
    norms = torch.empty((B,), device=dev)
    med_n, best_n = time_each(torch, lambda i: pe.pe_example_sqnorms(li.X, li.dY, norms))
    extra["pe_example_sqnorms_us"] = {"median": med_n * 1e3, "best": best_n * 1e3, "tflops_median": flops_one / med_n / 1e9}
    med_t, best_t = time_each(torch, lambda i: pe.pe_token_sqstats(li.X, li.dY, st["tok"]))
    extra["pe_token_sqstats_us"] = {"median": med_t * 1e3, "best": best_t * 1e3, "tflops_median": flops_one / med_t / 1e9}
    need = pe.pe_token_sqstats_staged_workspace_bytes(B, T, d_in, d_out)
    if need > 0:
        ws = st["tok_ws"] if st["tok_ws"] is not None else torch.empty(need, dtype=torch.uint8, device=dev)
        med_t2, best_t2 = time_each(torch, lambda i: pe.pe_token_sqstats_staged(li.X, li.dY, st["tok"], ws))
        extra["pe_token_sqstats_staged_us"] = {"median": med_t2 * 1e3, "best": best_t2 * 1e3, "tflops_median": flops_one / med_t2 / 1e9,
                                               "workspace_bytes": need}
        del ws
    need8 = pe.pe_token_sqstats_fp8_workspace_bytes(B, T, d_in, d_out)
    if need8 > 0 and d_in % 16 == 0 and d_out % 16 == 0:
        ws8 = torch.empty(need8, dtype=torch.uint8, device=dev)
        med_t8, best_t8 = time_each(torch, lambda i: pe.pe_token_sqstats_fp8(li.X, li.dY, st["tok"], ws8))
        extra["pe_token_sqstats_fp8_us"] = {"median": med_t8 * 1e3, "best": best_t8 * 1e3, "tflops_median": flops_one / med_t8 / 1e9,
                                            "note": "e4m3 operands: an approximation above the 2e-3 parity bound, not part of the timed step"}
        del ws8
    # statistics and parameter update in one launch, against the separate calls they replace
    fws = torch.empty(pe.pe_linear_fused_workspace_bytes(d_in, d_out), dtype=torch.uint8, device=dev)
    med_fa, best_fa = time_each(torch, lambda i: pe.pe_linear_microadam_step(li.X, li.dY, st["theta"], st["m"], st["v"], step=i + 1, theta_lp=st["theta_lp"],
                                                                             out_mean=st["mean"], out_stat=st["sq"], workspace=fws, **ADAM))
    med_ua, _ = time_each(torch, lambda i: pe.microadam_step(st["theta"], st["m"], st["v"], st["mean"], st["sq"], B, step=i + 1, theta_lp=st["theta_lp"], **ADAM))
    extra["pe_linear_microadam_step_us"] = {"median": med_fa * 1e3, "best": best_fa * 1e3, "separate_calls_median": (med + med_ua) * 1e3}
    med_fs, best_fs = time_each(torch, lambda i: pe.pe_linear_microsignsgd_step(li.X, li.dY, st["theta2"], st["m2"], theta_lp=st["theta2_lp"],
                                                                                out_sign=st["sgn"], workspace=fws, **SIGN))
    med_us, _ = time_each(torch, lambda i: pe.microsignsgd_step(st["theta2"], st["m2"], st["sgn"], B, theta_lp=st["theta2_lp"], **SIGN))
    extra["pe_linear_microsignsgd_step_us"] = {"median": med_fs * 1e3, "best": best_fs * 1e3, "separate_calls_median": (med_s + med_us) * 1e3}
    med_c, best_c = time_each(torch, lambda i: pe.pe_linear_clipped_sum(li.X, li.dY, 1.0, None, st["mean"]))
    extra["pe_linear_clipped_sum_us"] = {"median": med_c * 1e3, "best": best_c * 1e3, "note": "norms pass + scaled contraction"}
    del fws
    A2, B2 = li.dY.view(B * T, d_out), li.X.view(B * T, d_in)
    med_g, best_g = time_each(torch, lambda i: torch.matmul(A2.t(), B2))
    extra["cublas_wgrad_gemm_us"] = {"median": med_g * 1e3, "best": best_g * 1e3, "tflops_median": flops_one / med_g / 1e9,
                                     "note": "torch.matmul(dY_flat^T, X_flat), bf16 in and out"}
    extra["overhead_vs_gemm"] = med / med_g
    extra["overhead_all_three_vs_gemm"] = med_a3 / med_g
    big = 1 << 26       # update kernels on a parameter count far larger than L2 (64 Mi parameters)
    bufs = [torch.zeros(big, device=dev) for _ in range(5)]
    lp = torch.empty(big, dtype=torch.bfloat16, device=dev)
    med_a, _ = time_each(torch, lambda i: pe.microadam_step(bufs[0], bufs[1], bufs[2], bufs[3], bufs[4], B, step=1, theta_lp=lp, **ADAM), iters=10)
    med_sg, _ = time_each(torch, lambda i: pe.microsignsgd_step(bufs[0], bufs[1], bufs[3], B, theta_lp=lp, **SIGN), iters=10)
    extra["microadam_step"] = {"params": big, "gbs": 34.0 * big / med_a / 1e6, "frac_of_hbm_peak": 34.0 * big / med_a / 1e6 / peaks["hbm_gbs"]}
    extra["microsignsgd_step"] = {"params": big, "gbs": 22.0 * big / med_sg / 1e6, "frac_of_hbm_peak": 22.0 * big / med_sg / 1e6 / peaks["hbm_gbs"]}
    return extra


def run_sweep(args):
    """Shape sweep of a single bf16 layer (d_in = d_out): one JSON line per point with the time of
    pe_linear_stats(square, both outputs), of the statistic alone, and of the cuBLAS batch
    weight-gradient GEMM of the same shape."""
    import torch
    import paper_2510_00236_b200 as pe
    from paper_2510_00236_b200 import inputs
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pe.load_library()
    peaks = measured_peaks()
    for d in inputs.SWEEP_D:
        for (B, T) in inputs.SWEEP_BT:
            bytes_in = 2.0 * B * T * 2 * d
            nsets = max(1, min(6, int(300e6 // bytes_in)))      # rotate input sets until they exceed L2
            sets = [inputs.config5_point(B, T, d, dev, seed=inputs.BASE_SEED + 5 + 97 * k) for k in range(nsets)]
            mean = torch.empty((d, d), device=dev)
            stat = torch.empty((d, d), device=dev)
            flops = 2.0 * B * T * d * d

            def rested(fn):
                # every timed group starts one second after the device went idle: the clock the power limit left behind
                # a heavy group otherwise carries over into the next one (short sequences ran 1.5x slower right after a
                # 17 ms point), and the GEMM, timed last, would always meet the hottest chip
                torch.cuda.synchronize()
                time.sleep(1.0)
                return time_each(torch, fn, iters=12)

            med_b, best_b = rested(lambda i: pe.pe_linear_stats(sets[i % nsets].X, sets[i % nsets].dY, pe.PHI_SQUARE, mean, stat))
            med_s, best_s = rested(lambda i: pe.pe_linear_stats(sets[i % nsets].X, sets[i % nsets].dY, pe.PHI_SQUARE, None, stat))
            sgn = torch.empty((d, d), device=dev)
            med_n, _ = rested(lambda i: pe.pe_linear_stats(sets[i % nsets].X, sets[i % nsets].dY, pe.PHI_SIGN, None, stat))
            med_a, _ = rested(lambda i: pe.pe_linear_stats_all(sets[i % nsets].X, sets[i % nsets].dY, mean, stat, sgn))
            med_g, best_g = rested(lambda i: torch.matmul(sets[i % nsets].dY.view(B * T, d).t(), sets[i % nsets].X.view(B * T, d)))
            status, detail = pe.pe_get_async_status(dev)
            assert status == 0, (status, detail)
            # bounds per point: tensor pipe, the fp32 epilogue (2 ops per example and output entry on
            # 128 lanes x 148 SMs, packed 2-wide at best), and HBM
            t_tensor = flops / (peaks["bf16_tflops"] * 1e12)
            t_hbm = (bytes_in + 8.0 * d * d) / (peaks["hbm_gbs"] * 1e9)
            t_alu = 2.0 * B * d * d / (148 * 128 * 1.965e9)
            # the sign statistic alone costs 2 fp32 instructions per entry (packed scale, saturating fma, packed add), 4 beside
            # the other two sums; and short sequences are bound by how many
            # per-example tiles tensor memory holds at once: an accumulator entry is occupied for one hand-off chain
            # (about 1.25 us, measured: stage full seen -> MMAs and commits issued -> epilogue read -> release), 65536 entries per SM
            t_alu_sign = 4.0 * B * d * d / (148 * 128 * 1.965e9)
            t_occupancy = B * float(d) * d / (148 * 65536) * 1.25e-6
            print(json.dumps({
                "sweep_point": {"B": B, "T": T, "d_in": d, "d_out": d}, "input_sets": nsets,
                "both_outputs_us": med_b * 1e3, "both_outputs_tflops": flops / med_b / 1e9,
                "both_outputs_frac_of_peak": flops / med_b / 1e9 / peaks["bf16_tflops"],
                "stat_only_us": med_s * 1e3, "stat_only_tflops": flops / med_s / 1e9,
                "sign_only_us": med_n * 1e3, "all_three_us": med_a * 1e3, "overhead_all_three_vs_gemm": med_a / med_g,
                "cublas_gemm_us": med_g * 1e3, "cublas_gemm_tflops": flops / med_g / 1e9,
                "overhead_both_vs_gemm": med_b / med_g, "overhead_stat_vs_gemm": med_s / med_g,
                "bound_tensor_us": t_tensor * 1e6, "bound_hbm_us": t_hbm * 1e6, "bound_alu_us": t_alu * 1e6, "bound_alu_sign_us": t_alu_sign * 1e6,
                "bound_tmem_occupancy_us": t_occupancy * 1e6, "peak_source": peaks["source"]}), flush=True)
            del sets, mean, stat, sgn
            torch.cuda.empty_cache()


def oracle_sample(inputs, workload, n_rows, n_cols):
    """Column-gathered sub-layer of the workload for the CPU oracle (full B and T)."""
    import numpy as np
    B, T, d_in, d_out, _ = WORKLOADS[workload]
    if workload == "c2":
        li = inputs.config2("cpu")
    else:   # a reduced-batch stand-in keeps host generation bounded
        li = inputs.heavy_tailed_layer(32, T, d_in, d_out, seed=inputs.BASE_SEED + 4, device="cpu", name="c4", with_weights=False)
    rows = list(np.linspace(0, d_out - 1, n_rows).astype(int)) if n_rows < d_out else list(range(d_out))
    cols = list(np.linspace(0, d_in - 1, n_cols).astype(int)) if n_cols < d_in else list(range(d_in))
    sub = li if (n_rows >= d_out and n_cols >= d_in) else inputs.gather_columns(li, rows, cols)
    return inputs.to_numpy_bits(sub.X), inputs.to_numpy_bits(sub.dY)


def time_oracle(Xh, dYh):
    import oracle
    B, T, ni = Xh.shape
    no = dYh.shape[2]
    t0 = time.perf_counter()
    st = oracle.linear_stats(Xh, dYh)
    oracle.token_sqstats(Xh, dYh)
    import numpy as np
    z = np.zeros((no, ni))
    oracle.microadam_step(z, z, z, st.sum_g, st.sum_g2, B, step=1, **ADAM)
    oracle.microsignsgd_step(z, z, st.sum_sign, B, **SIGN)
    dt = time.perf_counter() - t0
    flops = 2 * 2.0 * B * T * ni * no      # the oracle forms G_b once for every phi, plus the per-token contraction
    return dt, flops


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2510_00236_b200 import inputs
    B, T, d_in, d_out, _ = WORKLOADS[args.workload]
    n_rows, n_cols = min(d_out, 256), min(d_in, 256)
    Xh, dYh = oracle_sample(inputs, args.workload, n_rows, n_cols)
    for _ in range(max(1, min(args.warmup, 3))):
        time_oracle(Xh, dYh)
    t = 0.0
    flops = 0.0
    for _ in range(args.steps):
        dt, fl = time_oracle(Xh, dYh)
        t += dt
        flops += fl
    value = flops / t / 1e12
    sample = f"{n_rows}x{n_cols} of the {d_out}x{d_in} outputs, B={Xh.shape[0]}, T={T} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": B, "T": T, "d_in": d_in, "d_out": d_out, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="shape sweep (B, T, d) instead of the step benchmark; one JSON line per point")
    ap.add_argument("--quick", action="store_true", help="timed region only: skip the per-kernel context numbers and the CPU baseline")
    ap.add_argument("--single-calls", action="store_true",
                    help="after the timed region also run pe_linear_stats(square, both outputs) and pe_linear_stats(sign) twice each, "
                         "so that a profiler capture of the run contains those kernels")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
        return
    if args.sweep:
        run_sweep(args)
        return

    import torch
    import paper_2510_00236_b200 as pe
    from paper_2510_00236_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    pe.load_library()          # fails loudly when the CUDA library is missing

    name = args.workload
    B, T, d_in, d_out, nsets = WORKLOADS[name]
    st = make_state(pe, inputs, torch, name, dev)
    flops_one = 2.0 * B * T * d_in * d_out
    flops_step = 2.0 * flops_one      # two contractions per step: the per-example one (all three statistics) and the per-token one

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ------------------------------------------------------------ device-resident timing
    for i in range(args.warmup):
        run_step(pe, st, i)
    status, detail = pe.pe_get_async_status(dev)
    assert status == 0, f"device status {status}/{detail}"
    assert pe.pe_last_path() == pe.PATH_TENSOR, "tensor-core path did not run"
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    pe.pe_reset_launch_count()
    kernel_events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        run_step(pe, st, args.warmup + i, ev=kernel_events[i])
    t_end.record()
    barrier()
    launches = pe.pe_launch_count()
    ms_total = t_start.elapsed_time(t_end)
    clocks = sampler.stop() if rank == 0 else None
    # average duration of each statistics call inside the timed steps (events on the launching stream)
    call_ms = [statistics.fmean(ev[k].elapsed_time(ev[k + 1]) for ev in kernel_events) for k in range(2)]
    ms_total = max_over_ranks(torch, dist, ms_total, dev)
    ms_step = ms_total / args.steps
    value = replica_throughput(world, flops_step, ms_step)

    # ------------------------------------------------------------ end to end: host buffers in, statistics out
    e2e_steps = max(3, min(20, args.steps // 5))
    li0 = st["sets"][0]
    hX = torch.empty(li0.X.shape, dtype=li0.X.dtype, pin_memory=True).copy_(li0.X)
    hdY = torch.empty(li0.dY.shape, dtype=li0.dY.dtype, pin_memory=True).copy_(li0.dY)
    # two device-side input buffers: the upload of step i+1 (copy stream) overlaps the kernels of step i (the
    # stream the library is called on), as a training loop that prefetches its next batch would
    dbuf = [(torch.empty_like(li0.X), torch.empty_like(li0.dY)) for _ in range(2)]
    outs = [st["mean"], st["sq"], st["sgn"], st["tok"]]
    houts = [torch.empty(o.shape, dtype=o.dtype, pin_memory=True) for o in outs]
    main_stream = torch.cuda.current_stream(dev)
    copy_stream = torch.cuda.Stream(device=dev)
    uploaded = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def upload(i):
        k = i % 2
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[k])          # the step that last read this buffer has finished
            dbuf[k][0].copy_(hX, non_blocking=True)
            dbuf[k][1].copy_(hdY, non_blocking=True)
            uploaded[k].record(copy_stream)

    def e2e_step(i):
        k = i % 2
        upload(i + 1)                                     # next step's inputs, while this step computes
        main_stream.wait_event(uploaded[k])
        run_step(pe, st, i, X=dbuf[k][0], dY=dbuf[k][1])
        consumed[k].record(main_stream)
        for h, o in zip(houts, outs):
            h.copy_(o, non_blocking=True)

    for k in range(2):
        consumed[k].record(main_stream)
    upload(0)
    for i in range(2):
        e2e_step(i)
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record()
    for i in range(2, 2 + e2e_steps):
        e2e_step(i)
    main_stream.wait_stream(copy_stream)      # the region holds exactly e2e_steps uploads: the last prefetch is waited for
    eb.record()
    barrier()
    e2e_ms = ea.elapsed_time(eb)
    e2e_ms = max_over_ranks(torch, dist, e2e_ms, dev)
    e2e_value = replica_throughput(world, flops_step, e2e_ms / e2e_steps)
    h2d = hX.numel() * hX.element_size() + hdY.numel() * hdY.element_size()
    d2h = sum(o.numel() * o.element_size() for o in outs)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ------------------------------------------------------------ context numbers (rank 0, outside the timed region)
    peaks = measured_peaks()
    li = st["sets"][0]
    if args.single_calls:
        for _ in range(2):
            pe.pe_linear_stats(li.X, li.dY, pe.PHI_SQUARE, st["mean"], st["sq"])
            pe.pe_linear_stats(li.X, li.dY, pe.PHI_SIGN, None, st["sgn"])
        torch.cuda.synchronize()
    target = None if args.quick else target_call_numbers(torch, pe, st, li, peaks)
    extra = {} if args.quick else context_numbers(torch, pe, st, li, peaks, dev)

    # One roofline entry per statistics call of the step; the headline one is the per-example statistics
    # kernel (the kernel the throughput target is about).  A step of the large layer runs long enough to be
    # power-capped, so the fraction of the sustained peak is given beside the burst one.  The one-kernel
    # per-token route contracts tf32 operands: its peak is the measured bf16 peak times the nominal
    # tf32 : bf16 ratio (1/2).
    alg_bytes = 2.0 * B * T * (d_in + d_out)
    specs = [("tc_stats_kernel<mean + square + sign>", "all", peaks["bf16_tflops"], "bf16", alg_bytes + 12.0 * d_in * d_out),
             ("tok_sqstats_kernel", "token", 0.5 * peaks["bf16_tflops"], "tf32", alg_bytes + 4.0 * d_in * d_out)]
    if st["tok_ws"] is not None:      # two-pass form: three streaming kernels around the half contraction
        specs[1] = ("pe_token_sqstats_staged: column_max + square_to_half + tc_stats_kernel<identity, half> + unscale", "token_staged",
                    peaks["bf16_tflops"], "f16", alg_bytes + 4.0 * d_in * d_out)
    by_kernel = []
    for (kname, key, peak, op_dtype, nbytes), ms in zip(specs, call_ms):
        ach = flops_one / (ms * 1e-3) / 1e12
        by_kernel.append({"bound": "tensor", "kernel": kname, "operand_dtype": op_dtype, "achieved": ach, "peak": peak,
                          "unit": "TFLOP/s", "frac": ach / peak,
                          "frac_of_sustained_peak": ach / (peak * peaks["bf16_tflops_sustained"] / peaks["bf16_tflops"]),
                          "peak_source": peaks["source"] + (" bf16 (burst) x 0.5 nominal tf32 ratio" if op_dtype == "tf32" else " (burst)"),
                          "traffic": profile_traffic(name, key), "avg_launch_ms": ms, "share_of_step": ms / ms_step,
                          "algorithmic_flops_per_launch": flops_one, "algorithmic_bytes_per_launch": nbytes})
    roofline = dict(by_kernel[0])
    roofline["by_kernel"] = by_kernel

    cpu_baseline = None
    if not args.no_cpu_baseline and not args.quick and world == 1:
        import oracle
        if name == "c2":
            Xh, dYh = inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY)
            sample = "the full workload, once"
        else:
            # the benchmark's own inputs, column-gathered: every output entry depends on one column of dY
            # and one of X, so the oracle computes this block of the workload's outputs exactly
            nr, nc = min(d_out, 512), min(d_in, 512)
            rows = torch.linspace(0, d_out - 1, nr, device=dev).long()
            cols = torch.linspace(0, d_in - 1, nc, device=dev).long()
            Xh = inputs.to_numpy_bits(li.X.index_select(2, cols).cpu())
            dYh = inputs.to_numpy_bits(li.dY.index_select(2, rows).cpu())
            sample = f"{nr}x{nc} of the {d_out}x{d_in} outputs at full B={B}, T={T}, once"
        dt, fl = time_oracle(Xh, dYh)
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": sample, "seconds": dt}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": name, "B": B, "T": T, "d_in": d_in, "d_out": d_out,
                   "step": "pe_linear_stats_all(mean,square,sign)+" + ("pe_token_sqstats_staged" if st["tok_ws"] is not None else "pe_token_sqstats")
                           + "+microadam_step+microsignsgd_step",
                   "flops_per_step": flops_step, "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": f"{nsets} rotating input sets, {nsets * 2 * B * T * (d_in + d_out) / 1e6:.0f} MB in all (> 126 MB L2)"
                         if nsets > 1 else "inputs larger than L2"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "pe_linear_stats": target,
        "cpu_baseline": cpu_baseline,
        "extra": extra,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
