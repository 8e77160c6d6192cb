#!/usr/bin/env python
"""Benchmark of the pQuant decoupled linear layer.

Metric: pQuant linear fwd+bwd tokens/s and fraction of the tensor-core roofline; decode GEMV fraction of HBM bandwidth.

One "step" of the headline = the whole training hot path over one batch of synthetic input: for each of the three
1.3B-shaped MLP projections (gate, up: 2048->5632; down: 5632->2048; 8192 tokens, HP width 128, one dense HP branch)
re-quantise the latent weights (pq_pack_weights), run pq_linear_forward and pq_linear_backward.

  python bench.py [--gpus N] [--steps K] [--warmup W]          # headline + sub-records (8 experts, decode, decoder step)
  python bench.py --workload mlp_dense|mlp_e8|decode|decoder   # one workload alone, with its own JSON line
  python bench.py --impl reference ...                          # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent replica of the workload on its own GPU --
the layer has no inter-GPU exchange -- and the slowest rank's time is used; `--gpus N` without a torchrun
environment re-launches itself under torch.distributed.run with N ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "pQuant linear fwd+bwd tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (the dW tiles of the 2048 -> 5632
# projection) from an ncu capture, stamped with the hash of the files that kernel is compiled from (the tensor-core engine,
# the GEMM kernels, the shared device helpers): once one of them changes the stamp no longer matches and the bench line
# reports null until the kernel is captured again.
NCU_TRAFFIC = {"bwd_dw": {"bytes": 218562048, "sources_sha16": "e1887889fce22bf8", "files": ("pq_gemm.cuh", "pq_gemm_kernels.cu", "pq_common.cuh")}}


def sources_sha16(files) -> str:
    """Hash of the named files of the library's source directory."""
    from paper_2602_22592_b200 import build as pqbuild
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(pqbuild.CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str):
    rec = NCU_TRAFFIC.get(kernel)
    return rec["bytes"] if rec and rec["sources_sha16"] == sources_sha16(rec["files"]) else None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def pick_bf16_peak(peaks, kind, timed_s, clocks):
    """The denominator that fits the timed region: the burst figure for a region shorter than about a second or run
    at (nearly) the maximum SM clock, the sustained one for a long region under the power cap."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    at_max = bool(mhz and mx and mhz >= 0.97 * mx)
    key = "bf16_tflops" if (timed_s < 1.0 or at_max) else "bf16_tflops_sustained"
    why = f"{kind} {key} (timed region {timed_s:.2f} s, median SM clock {mhz} of {mx} MHz)"
    return float(peaks[key]), key, why


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read only)."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self.nv:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- set-up shared by the GPU workloads
class Ctx:
    def __init__(self):
        import torch
        from paper_2602_22592_b200 import binding as pqb
        from paper_2602_22592_b200 import build as pqbuild
        from paper_2602_22592_b200 import replicas
        self.torch, self.pqb = torch, pqb
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
        torch.cuda.set_device(self.local)
        self.device = torch.device("cuda", self.local)
        self.reps = replicas.from_env("nccl", self.device)   # one replica per GPU, no collective on the data path
        self.world, self.rank = self.reps.world, self.reps.rank
        if self.rank == 0:
            pqbuild.build()
        self.reps.barrier()
        pqb.lib()
        self.peaks, self.peak_kind = measured_peaks()

    def barrier(self):
        self.reps.barrier()
        self.torch.cuda.synchronize()

    def check_status(self, what):
        code, where = self.pqb.pq_device_status()
        if code:
            raise RuntimeError(f"device-side wait timed out {what} (where={where})")


def measure_engine_peaks(ctx):
    """Rate of the library's own tensor-core engine on a plain 8192^3 contraction (raw accumulators written out),
    int8 (tcgen05 kind::i8) and bf16 (kind::f16): a measured lower bound of the int8 peak, which no library on the
    box reports, beside the same engine's bf16 rate for comparison with the cuBLAS figure."""
    torch, pqb = ctx.torch, ctx.pqb
    n = 8192
    out = {"shape": f"{n}^3, best of 10 launches, CUDA events"}
    gen = torch.Generator(device=ctx.device)
    gen.manual_seed(0)
    for mode, name, dt_in, dt_out in ((0, "i8_tops", torch.int8, torch.int32), (1, "bf16_tflops", torch.bfloat16, torch.float32)):
        if dt_in == torch.int8:
            A = torch.randint(-128, 128, (n, n), generator=gen, device=ctx.device, dtype=torch.int8)
            B = torch.randint(0, 2, (n, n), generator=gen, device=ctx.device, dtype=torch.int8) * 2 - 1
        else:
            A = torch.randn((n, n), generator=gen, device=ctx.device).to(dt_in)
            B = torch.randn((n, n), generator=gen, device=ctx.device).to(dt_in)
        D = torch.empty((n, n), dtype=dt_out, device=ctx.device)
        for _ in range(3):
            pqb.pq_debug_gemm(mode, n, n, n, A, B, D)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            pqb.pq_debug_gemm(mode, n, n, n, A, B, D)
            b.record()
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        out[name] = round(2.0 * n ** 3 / (best * 1e-3) / 1e12, 1)
        del A, B, D
    torch.cuda.empty_cache()
    return out


# --------------------------------------------------------------------------- training workloads (configs 2 and 3)
def build_mlp(E: int, device, T=None):
    from paper_2602_22592_b200 import inputs as I
    from paper_2602_22592_b200.layer import PQLinear
    cases = I.config_mlp(E, seed=1 if E == 1 else 2, T=T)
    layers = []
    for c in cases:
        L = PQLinear(c["T"], c["K"], c["N"], c["r"], c["E"], device=device).load_case(c)
        L.name = c["name"]
        layers.append(L)
    return layers, cases


def step_device(layers):
    for L in layers:
        L.pack()
        L.forward()
        L.backward()


def roofline_time_s(layers, p_bf16_tflops, p_i8_tops):
    """t_min = 2TNK / P_i8 + (4TNK + 6Tr(K+N)) / P_bf16 summed over the linears."""
    t = 0.0
    for L in layers:
        tnk = L.T * L.N * L.K
        t += 2 * tnk / (p_i8_tops * 1e12) + (4 * tnk + 6 * L.T * L.r * (L.K + L.N)) / (p_bf16_tflops * 1e12)
    return t


# algorithmic HBM bytes per launch of the memory-bound kernels, for the GB/s column of the breakdown
def elementwise_bytes(L, routed):
    T, K, N = L.T, L.K, L.N
    return {"pack_sums": 4 * N * K, "binarize_pack": 4 * N * K + N * K + N * K // 8,
            "act_quant": 2 * T * K + T * K + 2 * T * K + (2 * T * K if routed else 0),
            "router": 2 * T * K, "scatter_rows": 4 * T * N, "scaled_sign": N * K + 2 * N * K}


def measure_mlp(ctx, E, steps, warmup, engine, full):
    """Pack + forward + backward of the three MLP projections.  full: also the concurrent-stream figure, the
    per-kernel breakdown and the end-to-end leg."""
    torch, pqb, reps, device = ctx.torch, ctx.pqb, ctx.reps, ctx.device
    layers, cases = build_mlp(E, device)
    tokens = layers[0].T
    for _ in range(warmup):
        step_device(layers)
    ctx.barrier()
    ctx.check_status("during warm-up")

    # dominant kernel: the dW GEMM (contraction over tokens), timed live with events on the launch stream
    kid = pqb.KERNEL_IDS["bwd_dw"]
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers] for _ in range(steps)]
    for row in ev:
        for a, b in row:
            a.record(); b.record()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = pqb.pq_kernel_launches()
    ctx.barrier()
    with ClockSampler(ctx.local) as clk:
        t0.record()
        for s in range(steps):
            for i, L in enumerate(layers):
                L.pack()
                L.forward()
                pqb.pq_profile_events(kid, *ev[s][i])
                L.backward()
        t1.record()
        ctx.barrier()
    pqb.pq_profile_events(kid, None, None)
    launches = pqb.pq_kernel_launches() - launches0
    elapsed_ms = reps.max_over_ranks(t0.elapsed_time(t1), device)
    ctx.check_status("in the timed region")
    ms_per_step = elapsed_ms / steps
    clocks = clk.summary()
    peak, peak_key, peak_why = pick_bf16_peak(ctx.peaks, ctx.peak_kind, elapsed_ms * 1e-3, clocks)

    dw_ms = float(np.mean([a.elapsed_time(b) for row in ev for a, b in row]))
    # algorithmic flops of the launch: dW = dY^T . (q/gamma).  (The HP tiles dB, dA and the router gradient are a
    # launch of their own, profile id hp_db, and are not counted here.)  The launch shares the GPU with the chain
    # scaled sign -> HP gradient GEMM -> dX on the library's helper stream, so its event time includes SMs it
    # had to wait for.
    dw_flops = float(np.mean([2.0 * L.T * L.N * L.K for L in layers]))
    achieved = dw_flops / (dw_ms * 1e-3) / 1e12
    roofline = {"kernel": "k_gemm_bwd_dw (dW = dY^T . q/gamma, bf16 tcgen05, fp32 accumulate)", "bound": "tensor",
                "achieved": round(achieved, 1), "peak": peak, "unit": "TFLOP/s", "frac": round(achieved / peak, 4),
                "peak_source": peak_why, "avg_launch_ms": round(dw_ms, 4),
                "frac_of_burst": round(achieved / ctx.peaks["bf16_tflops"], 4),
                "frac_of_sustained": round(achieved / ctx.peaks["bf16_tflops_sustained"], 4),
                "traffic": ncu_traffic("bwd_dw")}
    mhz = clocks.get("sm_mhz") or 0.0
    # layer level: the int8 term at the nominal ratio 2 x bf16 (no library on the box measures an int8 peak) and, beside
    # it, at the rate this library's own engine reaches on a plain int8 contraction (a measured lower bound)
    t_nom = roofline_time_s(layers, peak, 2 * peak)
    layer = {"t_min_ms": round(t_nom * 1e3, 4), "frac": round(t_nom / (ms_per_step * 1e-3), 4),
             "formula": f"2TNK/P_i8 + (4TNK + 6Tr(K+N))/P_bf16, P_bf16 = {peak_key}, P_i8 = 2 P_bf16 (nominal ratio)",
             "ms_x_sm_mhz": round(ms_per_step * mhz, 1)}
    if engine:
        t_meas = roofline_time_s(layers, peak, engine["i8_tops"])
        layer["frac_with_measured_i8"] = round(t_meas / (ms_per_step * 1e-3), 4)
        layer["p_i8_measured_tops"] = engine["i8_tops"]
    rec = {"ms_per_step": round(ms_per_step, 4), "value": round(reps.whole_job_rate(tokens, ms_per_step), 1), "unit": "tokens/s",
           "steps": steps, "roofline": roofline, "layer_roofline": layer, "gpu_launches": int(launches), "clocks": clocks,
           "tokens": tokens, "experts": E}
    if not full:
        return rec, layers, cases

    # The same step with each projection's pack + forward + backward on a stream of its own (the three linears are
    # independent): tails of one projection's kernels and its memory-bound kernels overlap the others' GEMMs.
    # Reported beside the headline, which stays the single-stream figure the roofline numbers belong to.
    n_conc = max(3, min(steps, 50))
    side = [torch.cuda.Stream(device=device) for _ in layers]
    main_stream = torch.cuda.current_stream(device)

    def step_concurrent():
        fork = torch.cuda.Event()
        fork.record(main_stream)
        for L, st in zip(layers, side):
            st.wait_event(fork)
            with torch.cuda.stream(st):
                L.pack()
                L.forward()
                L.backward()
            done = torch.cuda.Event()
            done.record(st)
            main_stream.wait_event(done)

    for _ in range(2):
        step_concurrent()
    ctx.barrier()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(n_conc):
        step_concurrent()
    c1.record()
    ctx.barrier()
    conc_ms = reps.max_over_ranks(c0.elapsed_time(c1), device) / n_conc
    rec["concurrent_streams"] = {"streams": len(side), "steps": n_conc, "ms_per_step": round(conc_ms, 4),
                                 "value": round(reps.whole_job_rate(tokens, conc_ms), 1), "unit": "tokens/s",
                                 "note": "each projection on its own stream; not the headline"}
    rec["breakdown_us_per_step"], rec["elementwise_gbs"] = breakdown(ctx, layers, E > 1)
    return rec, layers, cases


def breakdown(ctx, layers, routed):
    """Per-kernel device time: mean over a few extra (untimed) steps, every kernel on one stream (helper stream off) so
    that each pair of events brackets one kernel running alone; the weight gradient is then a single launch again.
    Second result: achieved GB/s of the memory-bound kernels over their algorithmic bytes."""
    torch, pqb = ctx.torch, ctx.pqb
    pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 0)
    names = ["pack_sums", "binarize_pack", "router", "route_scan", "act_quant", "hp_up", "fwd", "scatter_rows", "scaled_sign",
             "hp_dh", "bwd_dx", "bwd_dw", "hp_db", "sum_partials", "sum_scalar"]
    bev = {n: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for n in names}
    total = {n: 0.0 for n in names}
    algo = {}
    bsteps = 5
    for _ in range(bsteps):
        for L in layers:
            for n, (a, b) in bev.items():
                a.record(); b.record()
                pqb.pq_profile_events(pqb.KERNEL_IDS[n], a, b)
            L.pack(); L.forward(); L.backward()
            torch.cuda.synchronize()
            for n, (a, b) in bev.items():
                total[n] += a.elapsed_time(b) * 1e3 / bsteps
    for L in layers:
        for n, by in elementwise_bytes(L, routed).items():
            algo[n] = algo.get(n, 0) + by
    for n in names:
        pqb.pq_profile_events(pqb.KERNEL_IDS[n], None, None)
    pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 1)
    # an id that was not launched shows only the few microseconds between its two back-to-back records
    out = {n: round(v, 1) for n, v in total.items() if v > 8.0 * len(layers)}
    gbs = {n: round(algo[n] / (out[n] * 1e-6) / 1e9, 0) for n in algo if n in out}
    return out, gbs


def measure_e2e_mlp(ctx, layers, steps):
    """End to end: inputs come from pinned host memory and results go back, every step."""
    torch, reps, device = ctx.torch, ctx.reps, ctx.device
    tokens = layers[0].T
    hx = [L.X.cpu().pin_memory() for L in layers]
    hdy = [L.dY.cpu().pin_memory() for L in layers]
    hy = [torch.empty_like(L.Y, device="cpu").pin_memory() for L in layers]
    hdx = [torch.empty_like(L.dX, device="cpu").pin_memory() for L in layers]
    # Copies and kernels on three streams: while projection i computes, the inputs of projection i + 1 come in
    # and the results of projection i - 1 go out (PCIe is full duplex).  Events keep a buffer from being
    # overwritten before its last reader is done.
    s_comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    ev_in = [torch.cuda.Event() for _ in layers]
    ev_comp = [torch.cuda.Event() for _ in layers]
    ev_out = [torch.cuda.Event() for _ in layers]
    for e in ev_in + ev_comp + ev_out:
        e.record(s_comp)

    def step_e2e():
        for i, L in enumerate(layers):
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_comp[i])              # the previous step's kernels have read X, dY
                L.X.copy_(hx[i], non_blocking=True)
                L.dY.copy_(hdy[i], non_blocking=True)
                ev_in[i].record(s_in)
            s_comp.wait_event(ev_in[i])
            s_comp.wait_event(ev_out[i])                 # the previous step's Y, dX have left
            L.pack(); L.forward(); L.backward()
            ev_comp[i].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[i])
                hy[i].copy_(L.Y, non_blocking=True)
                hdx[i].copy_(L.dX, non_blocking=True)
                ev_out[i].record(s_out)

    def drain():
        for e in ev_out:
            s_comp.wait_event(e)

    n_e2e = max(3, min(steps, 10))
    for _ in range(2):
        step_e2e()
    drain()
    ctx.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(n_e2e):
        step_e2e()
    drain()
    t1.record()
    ctx.barrier()
    ms = reps.max_over_ranks(t0.elapsed_time(t1), device)
    bi = sum(t.numel() * t.element_size() for t in hx + hdy)
    bo = sum(t.numel() * t.element_size() for t in hy + hdx)
    return {"value": round(reps.whole_job_rate(tokens, ms / n_e2e), 1), "unit": "tokens/s", "h2d_bytes_per_step": bi,
            "d2h_bytes_per_step": bo, "steps": n_e2e,
            "note": "X and dY of each projection copied from pinned host memory, Y and dX copied back, copies on their own streams overlapping the kernels; weights stay resident"}


WORKLOAD_TEXT = {
    1: "1.3B LLaMA MLP projections gate/up/down as pQuant linears, 8192 tokens, hidden 2048, FFN 5632, HP width 128, 1 expert(s)",
    8: "1.3B LLaMA MLP projections gate/up/down as pQuant linears, 8192 tokens, hidden 2048, FFN 5632, HP width 128, 8 expert(s), Zipf(1.1) routing",
}


def run_mlp(args, ctx, with_subrecords):
    E = 8 if args.workload == "mlp_e8" else 1
    engine = measure_engine_peaks(ctx)
    rec, layers, cases = measure_mlp(ctx, E, args.steps, args.warmup, engine, full=True)
    e2e = None if args.no_e2e else measure_e2e_mlp(ctx, layers, args.steps)
    del layers
    ctx.torch.cuda.empty_cache()
    cpu_baseline = None
    if ctx.rank == 0 and ctx.world == 1 and not args.no_cpu:
        cpu_baseline = oracle_baseline(E, sample_tokens=args.cpu_tokens)
    sub = {}
    if with_subrecords and ctx.world == 1:
        sub = subrecords(args, ctx, engine)
    if ctx.rank == 0:
        out = {
            "metric": METRIC, "value": rec["value"], "unit": "tokens/s", "n_gpus": ctx.world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x int8 -> int32 (forward 1-bit branch); bf16 -> fp32 (HP branch, backward)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[E], "tokens_per_step": rec["tokens"],
                       "l2": "inputs larger than L2 (each projection moves > 400 MB per step)", "replicas": ctx.world},
            "roofline": rec["roofline"], "layer_roofline": rec["layer_roofline"], "engine_peaks": engine,
            "breakdown_us_per_step": rec["breakdown_us_per_step"], "elementwise_gbs": rec["elementwise_gbs"],
            "concurrent_streams": rec["concurrent_streams"],
            "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": rec["gpu_launches"], "clocks": rec["clocks"],
        }
        out.update(sub)
        print(json.dumps(out))
    ctx.reps.close()


def subrecords(args, ctx, engine):
    """The rest of the metric in the same line: the routed training configuration, the decode path at M = 1, 4, 16
    (fraction of the HBM rate) and the whole-decoder step.  Short step counts; a failure is recorded, not raised."""
    out = {}
    torch = ctx.torch

    def guarded(name, fn):
        try:
            out[name] = fn()
        except Exception as e:   # noqa: BLE001 -- the headline must survive a failing sub-record
            out[name] = {"error": f"{type(e).__name__}: {e}"[:300]}
        torch.cuda.empty_cache()

    def e8():
        rec, layers, _ = measure_mlp(ctx, 8, max(10, min(args.steps, 50)), 3, engine, full=True)
        del layers
        keep = ("value", "unit", "ms_per_step", "steps", "layer_roofline", "roofline", "breakdown_us_per_step", "elementwise_gbs", "clocks")
        r = {k: rec[k] for k in keep}
        r["workload"] = WORKLOAD_TEXT[8]
        return r

    guarded("mlp_e8", e8)
    if not args.no_decode:
        def dec():
            weights = build_decode_weights(ctx)
            r = {"workload": decode_workload_text(None, False), "note": (
                "fraction of the measured HBM rate = algorithmic bytes / time / hbm_gbs.  batched16: 16 independent linears per "
                "launch (other sequences, parallel projections), one cooperative streaming kernel on weights in its own layout; "
                "batched_all: all 78 linears of the step handed to one pq_decode_batch call (one launch: the kernel's fixed costs -- "
                "token work, grid barrier, launch gap -- are paid once); "
                "pairs: what one sequence's model allows (gate + up of a block together); serial: one call per linear, each after "
                "the previous one -- both on the two-kernel path, which the library picks for small groups"),
                "kernels": ctx.decode_kernels}
            for M in (1, 4, 16):
                d = measure_decode(ctx, M, max(5, min(args.steps, 20)), weights, full=True)
                r[f"m{M}"] = {"batched16": d["batched"], "batched_all": d["batched_all"], "pairs": d["pairs"], "serial": d["serial"],
                              "algorithmic_bytes_per_step": d["algo"], "clocks": d["clocks"]}
            return r
        guarded("decode", dec)
    if not args.no_decoder:
        guarded("decoder", lambda: measure_decoder(ctx, max(2, min(args.steps, 5)), 3, True, engine))
    return out


# --------------------------------------------------------------------------- decode workload (config 5)
DECODE_LAYERS = 26   # depth of the 3B-shaped decoder whose MLP projections form the working set


def decode_workload_text(M, rmsnorm):
    from paper_2602_22592_b200 import inputs as I
    hid, ffn, r, E = I.DECODE_3B["hidden"], I.DECODE_3B["ffn"], I.DECODE_3B["r"], I.DECODE_3B["E"]
    m = "M in {1, 4, 16} tokens" if M is None else f"{M} token(s)"
    return (f"decode, {m}: {DECODE_LAYERS} layers x gate/up/down of a 3B-shaped model (hidden {hid}, FFN {ffn}), "
            f"1-bit weights packed 32 per word, {E} bf16 experts of width {r}, top-1, Zipf(1.1)"
            + (", RMSNorm fused in front of the quantiser" if rmsnorm else ""))


def build_decode_weights(ctx):
    """78 distinct weight sets (far more bytes than L2), drawn on the device (N(0, 0.02), the same law as the host
    generator: 78 host draws of 27.6 M normals would dominate the run), packed, latent copies dropped."""
    torch, device = ctx.torch, ctx.device
    from paper_2602_22592_b200 import inputs as I
    from paper_2602_22592_b200.layer import PQLinear
    hid, ffn, r, E = I.DECODE_3B["hidden"], I.DECODE_3B["ffn"], I.DECODE_3B["r"], I.DECODE_3B["E"]
    gen = torch.Generator(device=device)
    gen.manual_seed(4)
    sets = []
    for layer in range(DECODE_LAYERS):
        for i, (name, K, N) in enumerate(I.mlp_shapes(hid, ffn)):
            L = PQLinear(1, K, N, r, E, device=device, training=False)
            L.W = torch.randn((N, K), generator=gen, device=device, dtype=torch.float32) * 0.02
            L.pack(bits_only=True)
            sets.append(dict(K=K, N=N, r=r, E=E, seed=4 * 1024 + layer * 4 + i, w_bits=L.w_bits, w_scales=L.w_scales,
                             A=(torch.randn((E, r, K), generator=gen, device=device) * 0.02).to(torch.bfloat16),
                             B=(torch.randn((E, N, r), generator=gen, device=device) * 0.02).to(torch.bfloat16),
                             norm_weight=(1.0 + 0.1 * torch.randn((K,), generator=gen, device=device)).to(torch.bfloat16)))
            # the same weights in the streaming decode kernel's layout (one-time, like the pack itself)
            L.B = sets[-1]["B"]
            L.pack_decode()
            sets[-1]["w_bits_il"], sets[-1]["B_il"] = L.w_bits_il, L.B_il
            if ctx.decode_hp8:
                # the INT8 high-precision branch: int8 codes of the experts, B8 in the streaming layout
                L.A = sets[-1]["A"]
                L.pack_decode_hp8()
                sets[-1]["A8"], sets[-1]["B8_il"], sets[-1]["hp_scales"] = L.A8, L.B8_il, L.hp_scales
            del L
    torch.cuda.synchronize()
    return sets


def make_decode_layers(ctx, M, weights, rmsnorm=False):
    torch, device = ctx.torch, ctx.device
    from paper_2602_22592_b200 import inputs as I
    from paper_2602_22592_b200.layer import PQLinear
    layers = []
    for w in weights:
        L = PQLinear(M, w["K"], w["N"], w["r"], w["E"], device=device, training=False)
        act = I.decode_activations(M, w["K"], w["E"], seed=w["seed"])
        L.w_bits, L.w_scales, L.A, L.B = w["w_bits"], w["w_scales"], w["A"], w["B"]
        L.w_s8 = None
        if ctx.decode_kernels != "pair":
            L.w_bits_il, L.B_il = w["w_bits_il"], w["B_il"]
        if ctx.decode_hp8:
            L.A8, L.B8_il, L.hp_scales = w["A8"], w["B8_il"], w["hp_scales"]
        L.X = torch.from_numpy(act["X"]).to(device).to(torch.bfloat16)
        L.Wr = torch.from_numpy(act["Wr"]).to(device).to(torch.bfloat16)
        L.alpha = torch.full((1,), 2.0, device=device)
        L.beta = torch.full((1,), 0.2, device=device)
        if rmsnorm:
            L.norm_weight = w["norm_weight"]
            L.norm_eps = 1e-5
        layers.append(L)
    return layers


def measure_decode(ctx, M, steps, weights, full, batch=16, rmsnorm=False):
    """Decode linears from packed 1-bit weights, all with distinct weights, M tokens each, replayed as one CUDA graph.
    The figure of merit is the algorithmic bytes that must be read, per second, against the measured HBM rate."""
    torch, pqb, reps, device = ctx.torch, ctx.pqb, ctx.reps, ctx.device
    layers = make_decode_layers(ctx, M, weights, rmsnorm)
    E, r = weights[0]["E"], weights[0]["r"]

    def step():
        for L in layers:
            L.decode()

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    ctx.check_status("during warm-up")
    # algorithmic bytes of one pass: sign bits + scale, the experts the tokens really use, router, activations
    algo = 0
    for L in layers:
        experts = L.decode_view()["expert"].cpu().numpy()
        algo += L.N * L.K // 8 + 4 + len(set(experts.tolist())) * (1 if ctx.decode_hp8 else 2) * r * (L.K + L.N) + 2 * E * L.K + 2 * M * L.K + 2 * M * L.N
    keep = []

    def capture(b):
        """One CUDA graph of the whole pass.  b = 1: one call per linear, each after the previous one, as the layers of
        a decoder depend on each other.  b > 1: pq_decode_batch over groups of b consecutive linears, treated as
        independent (other sequences, parallel projections), so their weights stream back to back."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            if b <= 1:
                step()
            else:
                for i in range(0, len(layers), b):
                    items = pqb.make_decode_items([L.decode_entry() for L in layers[i:i + b]])
                    keep.append(items)
                    pqb.pq_decode_batch(items)
        return g

    def time_graph(g):
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return reps.max_over_ranks(a.elapsed_time(b) / steps, device)

    nlin = len(layers)
    hbm = ctx.peaks["hbm_gbs"]

    def figures(ms):
        return {"ms_per_step": round(ms, 4), "us_per_linear": round(ms * 1e3 / nlin, 3), "gbs": round(algo / (ms * 1e-3) / 1e9, 1),
                "hbm_frac": round(algo / (ms * 1e-3) / 1e9 / hbm, 4)}

    launches0 = pqb.pq_kernel_launches()
    graph = capture(batch)
    launches_per_step = pqb.pq_kernel_launches() - launches0
    out = {"algo": int(algo), "nlin": nlin, "launches_per_step": int(launches_per_step), "layers": layers}
    if full:
        out["serial"] = figures(time_graph(capture(1)))
        out["pairs"] = figures(time_graph(capture(2)))
        out["batched_all"] = figures(time_graph(capture(nlin)))
    with ClockSampler(ctx.local) as clk:
        ms = time_graph(graph)
    out["batched"] = figures(ms)
    out["ms_per_step"] = ms
    out["clocks"] = clk.summary()
    ctx.check_status("in the decode passes")
    return out


def run_decode(args, ctx):
    torch, pqb, reps = ctx.torch, ctx.pqb, ctx.reps
    from paper_2602_22592_b200 import inputs as I
    M = args.decode_tokens
    hid, ffn, r, E = I.DECODE_3B["hidden"], I.DECODE_3B["ffn"], I.DECODE_3B["r"], I.DECODE_3B["E"]
    weights = build_decode_weights(ctx)
    d = measure_decode(ctx, M, args.steps, weights, full=not args.decode_skip_serial, batch=args.decode_batch, rmsnorm=args.decode_rmsnorm)
    layers, nlin, ms_per_step = d["layers"], d["nlin"], d["ms_per_step"]
    # the same pass launched call by call (no graph), and end to end: every linear's activations from pinned host
    # memory, every result back
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hx = [L.X.cpu().pin_memory() for L in layers]
    hy = [torch.empty_like(L.Y, device="cpu").pin_memory() for L in layers]

    def step_e2e():
        for i, L in enumerate(layers):
            L.X.copy_(hx[i], non_blocking=True)
            L.decode()
            hy[i].copy_(L.Y, non_blocking=True)

    for _ in range(2):
        step_e2e()
    torch.cuda.synchronize()
    n_e2e = max(3, min(args.steps, 10))
    t0.record()
    for _ in range(n_e2e):
        step_e2e()
    t1.record()
    torch.cuda.synchronize()
    ms_e2e = t0.elapsed_time(t1) / n_e2e
    cpu_baseline = None
    if ctx.rank == 0 and ctx.world == 1 and not args.no_cpu:
        cpu_baseline = oracle_decode_baseline(M, hid, ffn, r, E)
    if ctx.rank == 0:
        b = d["batched"]
        out = {
            "metric": "pQuant decode linear (packed 1-bit weights) tokens/s", "value": round(reps.whole_job_rate(M * nlin, ms_per_step), 1),
            "unit": "token-linears/s", "n_gpus": ctx.world, "steps": args.steps, "warmup": 3,
            "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "s8 x s8 -> s32 (1-bit branch), " + ("s8 x s8 -> s32 (INT8 experts)" if ctx.decode_hp8 else "bf16 -> f32 (experts)"),
            "data": "synthetic",
            "config": {"workload": decode_workload_text(M, args.decode_rmsnorm),
                       "linears_per_step": nlin, "l2": f"{d['algo'] / 1e6:.0f} MB of distinct weights per step, larger than L2",
                       "launch": f"one CUDA graph per step, pq_decode_batch over groups of {args.decode_batch} independent linears",
                       "kernels": ctx.decode_kernels, "hp_branch": "int8" if ctx.decode_hp8 else "bf16", "replicas": ctx.world},
            "roofline": {"kernel": "decode kernels (all launches of a step)", "bound": "hbm", "achieved": b["gbs"],
                         "peak": ctx.peaks["hbm_gbs"], "unit": "GB/s", "frac": b["hbm_frac"],
                         "peak_source": f"{ctx.peak_kind} hbm_gbs", "algorithmic_bytes_per_step": d["algo"],
                         "us_per_linear": b["us_per_linear"], "traffic": None},
            "serial": d.get("serial"), "pairs": d.get("pairs"), "batched_all": d.get("batched_all"),
            "cpu_baseline": cpu_baseline,
            "e2e": {"value": round(reps.whole_job_rate(M * nlin, ms_e2e), 1), "unit": "token-linears/s",
                    "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in hx),
                    "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in hy), "steps": n_e2e},
            "gpu_launches": int(d["launches_per_step"] * args.steps), "clocks": d["clocks"],
        }
        print(json.dumps(out))
    reps.close()


# --------------------------------------------------------------------------- whole decoder step (config 4)
def measure_decoder(ctx, steps, warmup, both_attention_forms, engine):
    """One QAT step (forward + backward, no optimiser) of a 24-layer 1.3B-shaped decoder whose 168 projections are
    pQuant linears with 8 experts, top-1; token ids uniform over the vocabulary.  The device time of the pq_* calls is
    summed from CUDA events around them and reported apart from the rest (attention, norms, rotary embedding, LM head,
    loss: plain torch)."""
    torch = ctx.torch
    from paper_2602_22592_b200.decoder_harness import PQDecoder

    def one(attn_hp):
        m = PQDecoder(attn_hp=attn_hp, device=ctx.device)
        ids, tgt = m.random_batch()
        for _ in range(warmup):
            m.step(ids, tgt)
        torch.cuda.synchronize()
        ctx.check_status("during the decoder warm-up")
        m.timer.enabled = True
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(ctx.local) as clk:
            t0.record()
            for _ in range(steps):
                loss = m.step(ids, tgt)
            t1.record()
            torch.cuda.synchronize()
        ctx.check_status("in the decoder steps")
        total = t0.elapsed_time(t1) / steps
        pq_ms = m.timer.total_ms() / steps
        clocks = clk.summary()
        peak, peak_key, _ = pick_bf16_peak(ctx.peaks, ctx.peak_kind, total * steps * 1e-3, clocks)
        t_min = m.roofline_time_s(peak * 1e12, 2 * peak * 1e12)
        rec = {"ms_per_step": round(total, 2), "pq_linear_ms": round(pq_ms, 2), "rest_ms": round(total - pq_ms, 2),
               "tokens_per_s": round(m.T / (total * 1e-3), 1), "pq_linear_tokens_per_s": round(m.T / (pq_ms * 1e-3), 1),
               "pq_linear_roofline": {"t_min_ms": round(t_min * 1e3, 2), "frac": round(t_min / (pq_ms * 1e-3), 4),
                                      "formula": f"sum over 168 linears of 2TNK/P_i8 + (4TNK + 6Tr(K+N))/P_bf16, P_bf16 = {peak_key}, P_i8 = 2 P_bf16"},
               "loss": round(float(loss), 4), "steps": steps, "clocks": clocks}
        if engine:
            rec["pq_linear_roofline"]["frac_with_measured_i8"] = round(
                m.roofline_time_s(peak * 1e12, engine["i8_tops"] * 1e12) / (pq_ms * 1e-3), 4)
        del m
        torch.cuda.empty_cache()
        return rec

    out = {"workload": ("one QAT step of a 24-layer 1.3B-shaped LLaMA decoder (hidden 2048, 16 heads, FFN 5632, RMSNorm, RoPE, vocabulary "
                        "32000), batch 4 x 2048 tokens, every projection a pQuant linear (HP width 128, 8 experts, top-1, natural routing); "
                        "pq_* calls timed apart from the torch rest"),
           "all_projections_8_experts": one(True)}
    if both_attention_forms:
        out["attention_projections_pure_1bit"] = one(False)
    return out


def run_decoder(args, ctx):
    engine = measure_engine_peaks(ctx)
    rec = measure_decoder(ctx, args.steps, args.warmup, not args.decoder_one_form, engine)
    main = rec["all_projections_8_experts"]
    if ctx.rank == 0:
        out = {"metric": "pQuant decoder QAT step tokens/s (pQuant-linear time apart)", "value": main["tokens_per_s"], "unit": "tokens/s",
               "n_gpus": ctx.world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": main["ms_per_step"],
               "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": "int8 x int8 -> int32 / bf16 -> fp32 (pQuant linears); bf16 (torch rest)", "data": "synthetic",
               "config": {"workload": rec["workload"], "l2": "activations and weights of a step far exceed L2", "replicas": ctx.world},
               "engine_peaks": engine, "decoder": rec, "clocks": main["clocks"], "e2e": None, "gpu_launches": int(ctx.pqb.pq_kernel_launches())}
        print(json.dumps(out))
    ctx.reps.close()


# --------------------------------------------------------------------------- oracle (CPU) arm
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_step(cases, sample_tokens):
    """The oracle as it stands on the first `sample_tokens` tokens of each projection."""
    from oracle import pquant_oracle as O
    for c in cases:
        X, dY = c["X"][:sample_tokens], c["dY"][:sample_tokens]
        f = O.linear_forward(X, c["W"], c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])
        O.linear_backward(dY, X, f, c["A"], c["B"], c["Wr"], c["alpha"], c["beta"])


def sample_text(sample_tokens, full_tokens):
    return "the whole batch of 8192 tokens" if sample_tokens >= full_tokens else f"first {sample_tokens} of {full_tokens} tokens"


def oracle_baseline(E, sample_tokens):
    from paper_2602_22592_b200 import inputs as I
    cases = I.config_mlp(E, seed=1 if E == 1 else 2, T=sample_tokens)
    t = time.perf_counter()
    oracle_step(cases, sample_tokens)
    dt = time.perf_counter() - t
    return {"value": round(sample_tokens / dt, 1), "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{sample_text(sample_tokens, I.MLP_1P3B['T'])} through pack + forward + backward of the three projections, once ({dt:.1f} s)"}


def oracle_decode_baseline(M, hid, ffn, r, E):
    """The oracle's decode forward as it stands on one layer's three linears (weights packed beforehand, as on the GPU)."""
    from oracle import pquant_oracle as O
    from paper_2602_22592_b200 import inputs as I
    rng = np.random.default_rng(7)
    prepared = []
    for i, (_, K, N) in enumerate(I.mlp_shapes(hid, ffn)):
        W = (rng.standard_normal((N, K), dtype=np.float32) * np.float32(0.02))
        mu, lam = O.weight_scales(W)
        bits = O.pack_bits(O.binarize(W, mu))
        A = I.bf16_values(rng.standard_normal((E, r, K), dtype=np.float32) * np.float32(0.02))
        B = I.bf16_values(rng.standard_normal((E, N, r), dtype=np.float32) * np.float32(0.02))
        act = I.decode_activations(M, K, E, seed=9000 + i)
        prepared.append((act["X"], bits, lam, A, B, act["Wr"]))
    t = time.perf_counter()
    for X, bits, lam, A, B, Wr in prepared:
        O.decode_forward(X, bits, lam, A, B, Wr, 2.0, 0.2)
    dt = time.perf_counter() - t
    return {"value": round(M * len(prepared) / dt, 1), "unit": "token-linears/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": f"the three linears of one layer ({M} token(s) each, {dt:.1f} s), weights packed beforehand"}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the headline workload (every step the whole batch unless
    --cpu-tokens asks for a sample).  Rank 0 alone works and prints."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_22592_b200 import inputs as I
    E = 8 if args.workload == "mlp_e8" else 1
    T = args.cpu_tokens
    cases = I.config_mlp(E, seed=1 if E == 1 else 2, T=T)
    warm = min(args.warmup, 1)        # a CPU program has nothing to warm beyond its first touch of the data
    for _ in range(warm):
        oracle_step(cases, T)
    t = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(cases, T)
    dt = (time.perf_counter() - t) / max(args.steps, 1)
    value = round(T / dt, 1)
    sample = f"{sample_text(T, I.MLP_1P3B['T'])} per step"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", str(args.gpus))),
           "steps": args.steps, "warmup": warm, "ms_per_step": round(dt * 1e3, 2), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": WORKLOAD_TEXT[E], "tokens_per_step": T, "sample": sample},
           "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def relaunch_under_torchrun(n):
    """`--gpus N` (N > 1) given to a plain `python bench.py`: start N ranks of this same command line."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all", "mlp_dense", "mlp_e8", "decode", "decoder"],
                    help="all = the dense-HP MLP headline plus sub-records for the other configurations")
    ap.add_argument("--decode-tokens", type=int, default=1, choices=range(1, 17), metavar="M")
    ap.add_argument("--decode-skip-serial", action="store_true", help="time only the batched graph (shorter runs under a profiler)")
    ap.add_argument("--decode-batch", type=int, default=16, help="independent decode linears per pq_decode_batch call")
    ap.add_argument("--decode-kernels", default="auto", choices=["auto", "stream", "pair"],
                    help="auto: the library picks per launch group; stream: the cooperative streaming kernel wherever the items allow; "
                         "pair: the two-kernel path on the plain layout")
    ap.add_argument("--decode-interleave", type=int, default=1, choices=[0, 1, 2], help="streaming decode kernel: side-by-side walk of its two work lists (0 never, 1 auto, 2 always)")
    ap.add_argument("--decode-hp8", action="store_true", help="decode with the INT8 high-precision branch (int8 experts: half the expert bytes)")
    ap.add_argument("--decode-mma-from", type=int, default=5, help="streaming decode kernel: token groups of at least this size use the tensor-core bit product")
    ap.add_argument("--decode-prefetch", type=int, default=1, choices=[0, 1], help="streaming decode kernel: L2 prefetch of the sign bits during the token work")
    ap.add_argument("--decode-rmsnorm", action="store_true", help="decode from un-normalised activations, RMSNorm fused into the token preparation")
    ap.add_argument("--decoder-one-form", action="store_true", help="decoder workload: only the form with 8 experts on every projection")
    ap.add_argument("--cpu-tokens", type=int, default=8192, help="tokens per step of the CPU oracle (cpu_baseline and --impl reference)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="skip the decode sub-record of the default run")
    ap.add_argument("--no-decoder", action="store_true", help="skip the decoder-step sub-record of the default run")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_under_torchrun(args.gpus)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return
    ctx = Ctx()
    ctx.decode_kernels = args.decode_kernels
    ctx.decode_hp8 = args.decode_hp8
    ctx.pqb.pq_set_option(ctx.pqb.PQ_OPT_DECODE_INTERLEAVE, args.decode_interleave)
    ctx.pqb.pq_set_option(ctx.pqb.PQ_OPT_DECODE_STREAM, {"auto": 1, "stream": 2, "pair": 0}[args.decode_kernels])
    ctx.pqb.pq_set_option(ctx.pqb.PQ_OPT_DECODE_PREFETCH, args.decode_prefetch)
    ctx.pqb.pq_set_option(ctx.pqb.PQ_OPT_DECODE_MMA_FROM, args.decode_mma_from)
    if args.workload == "decode":
        run_decode(args, ctx)
    elif args.workload == "decoder":
        run_decoder(args, ctx)
    else:
        run_mlp(args, ctx, with_subrecords=args.workload == "all")


if __name__ == "__main__":
    main()
