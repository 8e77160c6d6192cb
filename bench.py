#!/usr/bin/env python
"""Benchmark of the pQuant decoupled linear layer (pack + forward + STE backward).

One "step" = the whole hot path over one batch of synthetic input: for each of
the three 1.3B-shaped MLP projections (gate, up: 2048->5632; down: 5632->2048;
8192 tokens, HP width 128) re-quantise the latent weights (pq_pack_weights),
run pq_linear_forward and pq_linear_backward.  Metric: tokens/s.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mlp_dense|mlp_e8|decode]
  python bench.py --impl reference ...      # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an
independent replica of the workload on its own GPU -- the layer has no
inter-GPU exchange -- and the slowest rank's time is used.
"""
from __future__ import annotations

import argparse
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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (the 2048 -> 5632
# projection) from the committed ncu capture (profiles/gemm_kernels_up_projection_ncu.md); set to None
# whenever the kernel changes until it is captured again.
NCU_TRAFFIC_BYTES = {"bwd_dw": 218165248}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


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


# --------------------------------------------------------------------------- workloads
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


def roofline_time_s(layers, peaks):
    """t_min = 2TNK / P_i8 + (4TNK + 6Tr(K+N)) / P_bf16 with P_i8 = 2 P_bf16 (nominal ratio)."""
    pb = peaks["bf16_tflops_sustained"] * 1e12
    t = 0.0
    for L in layers:
        tnk = L.T * L.N * L.K
        t += 2 * tnk / (2 * pb) + (4 * tnk + 6 * L.T * L.r * (L.K + L.N)) / pb
    return t


def run_ours(args):
    import torch
    from paper_2602_22592_b200 import binding as pqb
    from paper_2602_22592_b200 import build as pqbuild

    from paper_2602_22592_b200 import replicas
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    reps = replicas.from_env("nccl", device)   # one replica per GPU, no collective on the data path
    world, rank = reps.world, reps.rank
    if rank == 0:
        pqbuild.build()
    reps.barrier()
    pqb.lib()
    peaks, peak_kind = measured_peaks()

    E = 8 if args.workload == "mlp_e8" else 1
    layers, cases = build_mlp(E, device)
    tokens = layers[0].T

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step_device(layers)
    barrier()
    code, where = pqb.pq_device_status()
    if code:
        raise RuntimeError(f"device-side wait timed out during warm-up (where={where})")

    # dominant kernel: the dW GEMM (contraction over tokens), timed live with events on the launch stream
    kid = pqb.KERNEL_IDS["bwd_dw"]
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers] for _ in range(args.steps)]
    for row in ev:
        for a, b in row:
            a.record(); b.record()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = pqb.pq_kernel_launches()
    barrier()
    with ClockSampler(local) as clk:
        t0.record()
        for s in range(args.steps):
            for i, L in enumerate(layers):
                L.pack()
                L.forward()
                pqb.pq_profile_events(kid, *ev[s][i])
                L.backward()
        t1.record()
        barrier()
    pqb.pq_profile_events(kid, None, None)
    launches = pqb.pq_kernel_launches() - launches0
    elapsed_ms = reps.max_over_ranks(t0.elapsed_time(t1), device)
    code, where = pqb.pq_device_status()
    if code:
        raise RuntimeError(f"device-side wait timed out (where={where})")
    ms_per_step = elapsed_ms / args.steps
    value = reps.whole_job_rate(tokens, ms_per_step)

    dw_ms = float(np.mean([a.elapsed_time(b) for row in ev for a, b in row]))
    # algorithmic flops of the launch: dW = dY^T . (q/gamma).  (The HP tiles dB, dA and the router gradient are a
    # launch of their own, profile id hp_db, and are not counted here.)  The launch shares the GPU with the chain
    # scaled sign -> HP gradient GEMM -> dX on the library's helper stream, so its event time includes SMs it
    # had to wait for.
    dw_flops = float(np.mean([2.0 * L.T * L.N * L.K for L in layers]))
    achieved = dw_flops / (dw_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    roofline = {"kernel": "k_gemm_bwd_dw (dW = dY^T . q/gamma, bf16 tcgen05, fp32 accumulate)", "bound": "tensor",
                "achieved": round(achieved, 1), "peak": peak, "unit": "TFLOP/s", "frac": round(achieved / peak, 4),
                "peak_source": f"{peak_kind} bf16_tflops_sustained", "avg_launch_ms": round(dw_ms, 4),
                "traffic": NCU_TRAFFIC_BYTES["bwd_dw"]}
    t_min = roofline_time_s(layers, peaks)
    layer_frac = t_min / (ms_per_step * 1e-3)

    # The same step with each projection's pack + forward + backward on a stream of its own (the three linears are
    # independent): tails of one projection's kernels and its memory-bound kernels overlap the others' GEMMs.
    # Reported beside the headline, which stays the single-stream figure the roofline numbers belong to.
    n_conc = max(3, min(args.steps, 50))
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
    barrier()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(n_conc):
        step_concurrent()
    c1.record()
    barrier()
    conc_ms = reps.max_over_ranks(c0.elapsed_time(c1), device) / n_conc
    concurrent = {"streams": len(side), "steps": n_conc, "ms_per_step": round(conc_ms, 4),
                  "value": round(reps.whole_job_rate(tokens, conc_ms), 1), "unit": "tokens/s",
                  "note": "each projection on its own stream; not the headline"}

    # per-kernel breakdown: mean over a few extra (untimed) steps, every kernel on one stream (helper stream off) so
    # that each pair of events brackets one kernel running alone; the weight gradient is then a single launch again
    pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 0)
    names = ["pack_sums", "binarize_pack", "router", "route_scan", "act_quant", "hp_up", "fwd", "scatter_rows", "scaled_sign",
             "hp_dh", "bwd_dx", "bwd_dw", "hp_db", "reduce_db", "hp_da", "reduce_da", "router_wgrad", "sum_partials", "sum_scalar"]
    bev = {n: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for n in names}
    breakdown = {n: 0.0 for n in names}
    bsteps = 5
    for _ in range(bsteps):
        for L in layers:
            for n, (a, b) in bev.items():
                a.record(); b.record()
                pqb.pq_profile_events(pqb.KERNEL_IDS[n], a, b)
            l0 = pqb.pq_kernel_launches()
            L.pack(); L.forward(); L.backward()
            torch.cuda.synchronize()
            for n, (a, b) in bev.items():
                breakdown[n] += a.elapsed_time(b) * 1e3 / bsteps
    for n in names:
        pqb.pq_profile_events(pqb.KERNEL_IDS[n], None, None)
    pqb.pq_set_option(pqb.PQ_OPT_SIDE_STREAM, 1)
    # an id that was not launched shows only the few microseconds between its two back-to-back records
    breakdown = {n: round(v, 1) for n, v in breakdown.items() if v > 8.0 * len(layers)}

    # end to end: inputs come from pinned host memory and results go back, every step
    e2e = None
    if not args.no_e2e:
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

        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            step_e2e()
        drain()
        barrier()
        t0.record()
        for _ in range(n_e2e):
            step_e2e()
        drain()
        t1.record()
        barrier()
        ms = reps.max_over_ranks(t0.elapsed_time(t1), device)
        bi = sum(t.numel() * t.element_size() for t in hx + hdy)
        bo = sum(t.numel() * t.element_size() for t in hy + hdx)
        e2e = {"value": round(reps.whole_job_rate(tokens, ms / n_e2e), 1), "unit": "tokens/s", "h2d_bytes_per_step": bi,
               "d2h_bytes_per_step": bo, "steps": n_e2e,
               "note": "X and dY of each projection copied from pinned host memory, Y and dX copied back, copies on their own streams overlapping the kernels; weights stay resident"}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline = oracle_baseline(E, sample_tokens=args.cpu_tokens)

    if rank == 0:
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x int8 -> int32 (forward 1-bit branch); bf16 -> fp32 (HP branch, backward)",
            "data": "synthetic",
            "config": {"workload": ("1.3B LLaMA MLP projections gate/up/down as pQuant linears, 8192 tokens, hidden 2048, FFN 5632, "
                                    f"HP width 128, {E} expert(s)" + (", Zipf(1.1) routing" if E > 1 else "")),
                       "tokens_per_step": tokens, "l2": "inputs larger than L2 (each projection moves > 400 MB per step)",
                       "replicas": world},
            "roofline": roofline,
            "layer_roofline": {"t_min_ms": round(t_min * 1e3, 4), "frac": round(layer_frac, 4),
                               "formula": "2TNK/P_i8 + (4TNK + 6Tr(K+N))/P_bf16, P_i8 = 2 P_bf16, sustained bf16 peak"},
            "breakdown_us_per_step": breakdown, "concurrent_streams": concurrent,
            "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clk.summary(),
        }
        print(json.dumps(out))
    reps.close()


# --------------------------------------------------------------------------- decode workload
DECODE_LAYERS = 26   # depth of the 3B-shaped decoder whose MLP projections form the working set


def run_decode(args):
    """Decode linears from packed 1-bit weights: 26 layers x (gate, up, down) of a 3B-shaped model, all with
    distinct weights (far more bytes than L2), M tokens each, replayed as one CUDA graph.  The figure of merit
    is the algorithmic bytes of the weights that must be read, per second, against the measured HBM rate.
    Headline: the linears treated as independent and handed to pq_decode_batch in groups; beside it the same
    pass with one call per linear (dependent layers) and in groups of two."""
    import torch
    from paper_2602_22592_b200 import binding as pqb
    from paper_2602_22592_b200 import build as pqbuild
    from paper_2602_22592_b200 import inputs as I
    from paper_2602_22592_b200.layer import PQLinear

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    from paper_2602_22592_b200 import replicas
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    reps = replicas.from_env("nccl", device)   # one replica per GPU, no collective on the data path
    world, rank = reps.world, reps.rank
    if rank == 0:
        pqbuild.build()
    reps.barrier()
    pqb.lib()
    peaks, peak_kind = measured_peaks()
    M = args.decode_tokens
    hid, ffn, r, E = I.DECODE_3B["hidden"], I.DECODE_3B["ffn"], I.DECODE_3B["r"], I.DECODE_3B["E"]
    gen = torch.Generator(device=device)
    gen.manual_seed(4)
    layers = []
    for layer in range(DECODE_LAYERS):
        for i, (name, K, N) in enumerate(I.mlp_shapes(hid, ffn)):
            L = PQLinear(M, K, N, r, E, device=device, training=False)
            act = I.decode_activations(M, K, E, seed=4 * 1024 + layer * 4 + i)
            # weights drawn on the device (N(0, 0.02), the same law as the host generator), packed, latent copy dropped
            L.W = torch.randn((N, K), generator=gen, device=device, dtype=torch.float32) * 0.02
            L.pack(bits_only=True)
            L.W = None
            L.w_s8 = None
            L.A = (torch.randn((E, r, K), generator=gen, device=device) * 0.02).to(torch.bfloat16)
            L.B = (torch.randn((E, N, r), generator=gen, device=device) * 0.02).to(torch.bfloat16)
            L.X = torch.from_numpy(act["X"]).to(device).to(torch.bfloat16)
            L.Wr = torch.from_numpy(act["Wr"]).to(device).to(torch.bfloat16)
            L.alpha = torch.full((1,), 2.0, device=device)
            L.beta = torch.full((1,), 0.2, device=device)
            if args.decode_rmsnorm:
                L.norm_weight = (1.0 + 0.1 * torch.randn((K,), generator=gen, device=device)).to(torch.bfloat16)
                L.norm_eps = 1e-5
            layers.append(L)
    torch.cuda.synchronize()

    def step():
        for L in layers:
            L.decode()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    code, where = pqb.pq_device_status()
    if code:
        raise RuntimeError(f"device-side wait timed out during warm-up (where={where})")
    # algorithmic bytes of one pass: sign bits + scale, the experts the tokens really use, router, activations
    algo = 0
    for L in layers:
        experts = L.decode_view()["expert"].cpu().numpy()
        algo += L.N * L.K // 8 + 4 + len(set(experts.tolist())) * 2 * r * (L.K + L.N) + 2 * E * L.K + 2 * M * L.K + 2 * M * L.N
    def capture(batch):
        """One CUDA graph of the whole pass.  batch = 1: one call per linear, each after the previous one, as the
        layers of a decoder depend on each other.  batch > 1: pq_decode_batch over groups of `batch` consecutive
        linears, treated as independent (other sequences, parallel projections), so their weights stream back to back."""
        g = torch.cuda.CUDAGraph()
        keep = []
        with torch.cuda.graph(g):
            if batch <= 1:
                step()
            else:
                for i in range(0, len(layers), batch):
                    items = pqb.make_decode_items([L.decode_entry() for L in layers[i:i + batch]])
                    keep.append(items)
                    pqb.pq_decode_batch(items)
        return g

    def time_graph(g):
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return reps.max_over_ranks(a.elapsed_time(b) / args.steps, device)

    launches0 = pqb.pq_kernel_launches()
    graph = capture(args.decode_batch)
    launches_per_step = pqb.pq_kernel_launches() - launches0
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.decode_skip_serial:      # profiling runs: only the batched graph
        ms_serial = ms_pairs = float("nan")
    else:
        ms_serial = time_graph(capture(1))
        ms_pairs = time_graph(capture(2))
    with ClockSampler(local) as clk:
        ms_per_step = time_graph(graph)
    code, where = pqb.pq_device_status()
    if code:
        raise RuntimeError(f"device-side wait timed out (where={where})")
    # same pass launched call by call (no graph), for the launch-overhead comparison
    ms_eager = float("nan")
    if not args.decode_skip_serial:
        t0.record()
        for _ in range(min(args.steps, 20)):
            step()
        t1.record()
        torch.cuda.synchronize()
        ms_eager = t0.elapsed_time(t1) / min(args.steps, 20)

    # end to end: every linear's activations from pinned host memory, every result back
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

    gbs = algo / (ms_per_step * 1e-3) / 1e9
    nlin = len(layers)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline = oracle_decode_baseline(M, hid, ffn, r, E)
    if rank == 0:
        out = {
            "metric": "pQuant decode linear (packed 1-bit weights) tokens/s", "value": round(reps.whole_job_rate(M * nlin, ms_per_step), 1),
            "unit": "token-linears/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8 bit masks x s8 -> s32 (1-bit branch), bf16 -> f32 (experts)", "data": "synthetic",
            "config": {"workload": (f"decode, {M} token(s): {DECODE_LAYERS} layers x gate/up/down of a 3B-shaped model (hidden {hid}, FFN {ffn}), "
                                    f"1-bit weights packed 32 per word, {E} bf16 experts of width {r}, top-1, Zipf(1.1)"
                                    + (", RMSNorm fused in front of the quantiser" if args.decode_rmsnorm else "")),
                       "linears_per_step": nlin, "l2": f"{algo / 1e6:.0f} MB of distinct weights per step, larger than L2",
                       "launch": f"one CUDA graph per step, pq_decode_batch over groups of {args.decode_batch} independent linears", "replicas": world},
            "roofline": {"kernel": "k_decode_prep + k_decode_main (all launches of a step)", "bound": "hbm", "achieved": round(gbs, 1),
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
                         "peak_source": f"{peak_kind} hbm_gbs", "algorithmic_bytes_per_step": int(algo),
                         "us_per_linear": round(ms_per_step * 1e3 / nlin, 3), "traffic": None},
            "serial": {"ms_per_step": round(ms_serial, 4), "us_per_linear": round(ms_serial * 1e3 / nlin, 3),
                       "hbm_frac": round(algo / (ms_serial * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                       "note": "the same pass with one call per linear, each after the previous one has finished (dependent layers)"},
            "pairs": {"ms_per_step": round(ms_pairs, 4), "us_per_linear": round(ms_pairs * 1e3 / nlin, 3),
                      "hbm_frac": round(algo / (ms_pairs * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                      "note": "batches of two (what the gate and up projections of one block allow)"},
            "eager_ms_per_step": round(ms_eager, 4),
            "cpu_baseline": cpu_baseline,
            "e2e": {"value": round(reps.whole_job_rate(M * nlin, ms_e2e), 1), "unit": "token-linears/s",
                    "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in hx),
                    "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in hy), "steps": n_e2e},
            "gpu_launches": int(launches_per_step * args.steps), "clocks": clk.summary(),
        }
        print(json.dumps(out))
    reps.close()


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


def oracle_baseline(E, sample_tokens):
    from paper_2602_22592_b200 import inputs as I
    cases = I.config_mlp(E, seed=1 if E == 1 else 2, T=sample_tokens)
    t = time.perf_counter()
    oracle_step(cases, sample_tokens)
    dt = time.perf_counter() - t
    return {"value": round(sample_tokens / dt, 1), "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": (f"first {sample_tokens} of 8192 tokens through pack + forward + backward of the three projections "
                       f"({dt:.1f} s; the per-matrix weight quantisation does not shrink with the sample, so this understates "
                       "the full-batch rate)")}


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
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_22592_b200 import inputs as I
    E = 8 if args.workload == "mlp_e8" else 1
    T = args.cpu_tokens
    cases = I.config_mlp(E, seed=1 if E == 1 else 2, T=T)
    for _ in range(min(args.warmup, 1)):
        oracle_step(cases, T)
    steps = max(1, min(args.steps, 5))
    t = time.perf_counter()
    for _ in range(steps):
        oracle_step(cases, T)
    dt = (time.perf_counter() - t) / steps
    value = round(T / dt, 1)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": round(dt * 1e3, 2), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"1.3B LLaMA MLP projections as pQuant linears, {E} expert(s); CPU oracle on a {T}-token sample per step"},
           "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
                            "sample": f"{T} of 8192 tokens per step"},
           "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp_dense", choices=["mlp_dense", "mlp_e8", "decode"])
    ap.add_argument("--decode-tokens", type=int, default=1, choices=range(1, 17), metavar="M")
    ap.add_argument("--decode-skip-serial", action="store_true", help="time only the batched graph (shorter runs under a profiler)")
    ap.add_argument("--decode-batch", type=int, default=16, help="independent decode linears per pq_decode_batch call")
    ap.add_argument("--decode-rmsnorm", action="store_true", help="decode from un-normalised activations, RMSNorm fused into the token preparation")
    ap.add_argument("--cpu-tokens", type=int, default=4096)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "decode":
        run_decode(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
