"""Benchmark of the W4A8 quantized linear layer (FP4 weights, FP8 activations, LoRC) on B200.

A step is SWEEPS passes of the whole hot path (token-wise FP8 quantization with the LoRC down-projection,
then the W4A8 GEMM with its scale + LoRC epilogue) over the OPT-30B-shaped sweep: the two MLP layers
(7168 -> 28672 and 28672 -> 7168), each at M in {8192, 2048, 512, 128, 32, 8, 1} tokens, constraint M2,
group 128, LoRC rank 8.  Weights are packed once before the timed region.  A layer call is
zq_w4a8_linear on raw bf16 activations (the library quantizes: inside the GEMM kernel up to 16 tokens, with its
quantizer kernel chained to the GEMM beyond); the calls at the
largest token count are issued as quantizer call + GEMM call so that CUDA events can bracket the dominant
GEMM kernel inside the timed region.  The sweep runs from many tokens to few: a decode-size call right
after the 8192-token GEMM would be timed while that kernel's 235 MB of output is still being written back
from L2 (measured: 35 us instead of 27 us for the same launch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-cpu-baseline]

Prints one JSON line.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
With --gpus N > 1 outside a torchrun environment the script starts the N ranks itself.
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

from paper_2307_09782_b200 import synth  # noqa: E402

WORKLOAD = "opt30b"
GROUP, MODE, RANK = 128, "M2", 8
NOMINAL_FP8_TFLOPS = 4500.0  # public dense FP8 figure of the part, for context
# DRAM bytes per launch from the ncu captures summarised under profiles/ (null when the kernel changed since)
DOMINANT_TRAFFIC = 1760e6  # mean of the two M = 8192 launches (1516 MB and 2003 MB)
DECODE_TRAFFIC = 114.5e6   # 7168 -> 28672 at 8 tokens
# LLaMA-7B-shaped rows outside the timed step: (scale mode, weight layout)
EXTRA_LLAMA7B = (("none", "cast"), ("none", "mx"), ("M2", "mx"))
METRIC = "w4a8_linear_tflops"
UNIT = "TFLOP/s"
N_WEIGHT_COPIES = 2  # per layer; rotated so that > 2x the L2 size streams between two reads of one buffer


def flops(M, N, K, r):
    return 2.0 * M * N * K + 2.0 * M * r * (K + N)


def weight_bytes(N, K, group=GROUP):
    return N * K / 2 + N * K / group + 4 * N


def layer_bytes(M, N, K, r, group=GROUP):
    """Bytes the whole layer must move (M1 / M2, FP32 y): codes, shifts, channel scales, x, y, U, V."""
    return weight_bytes(N, K, group) + 2 * M * K + 4 * M * N + 2 * r * (N + K)


def gemm_bytes(M, N, K, r, group=GROUP):
    """Bytes of the GEMM alone on pre-quantized activations: weights, q, sx, t, y, U."""
    return weight_bytes(N, K, group) + M * K + 4 * M + 4 * M * r + 4 * M * N + 2 * r * N


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------------
def oracle_sample_step(wl, state=None, M_s=8):
    """One bounded sample of the workload on the host cores: the first M_s tokens of the first layer
    (quantizer + LoRC down-projection + all N outputs of the linear).  Returns (seconds, flops, state)."""
    import oracle

    shape = wl.shapes[0]
    if state is None:
        state = {}
        state["x"] = synth.make_x(wl.seed, M_s, shape.K, wl.n_outliers(shape.K), wl.outlier_factor)
        W = synth.make_w(wl.seed, shape.N, shape.K, wl.sigma_w)
        state["U"], state["V"] = synth.make_lorc(wl.seed, shape.N, shape.K, RANK)
        state["packed"] = oracle.pack_weight_fp4(W, GROUP, MODE)  # offline step, not timed
    t0 = time.perf_counter()
    q, sx, t = oracle.quantize_act_fp8(state["x"], state["V"])
    c, sh, sc = state["packed"]
    oracle.w4a8_linear(q, sx, c, sh, sc, GROUP, MODE, state["U"], t)
    dt = time.perf_counter() - t0
    return dt, flops(M_s, shape.N, shape.K, RANK), state


def base_config(args, shapes, Ms, mode):
    return {"workload": WORKLOAD if not args.case else f"case {args.case}",
            "layers": [f"{s.K}->{s.N}" for s in shapes], "M": Ms, "group": GROUP, "mode": mode,
            "weight_layout": args.layout, "lorc_rank": RANK,
            "launches": ("cooperative where CTAs share output tiles (library default)" if args.cooperative else
                         "plain: zq_set_exclusive_device(1), the bench has the device to itself")}


def cpu_baseline(wl):
    import oracle

    dt, fl, _ = oracle_sample_step(wl, M_s=32)
    shape = wl.shapes[0]
    return {"value": fl / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{wl.name} {shape.K}->{shape.N}: first 32 tokens, all {shape.N} outputs, quantizer + LoRC + "
                      f"FP64 linear, {dt:.1f} s"}


def run_reference(args):
    import oracle

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.WORKLOADS[WORKLOAD]
    state = None
    times, fl = [], 0.0
    for i in range(args.warmup + args.steps):
        dt, fl, state = oracle_sample_step(wl, state, M_s=2)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = fl * len(times) / total / 1e12
    shape = wl.shapes[0]
    sample = (f"each step: {wl.name} {shape.K}->{shape.N}, first 2 tokens, all outputs (quantizer + LoRC + FP64 "
              f"linear); a bounded sample of the sweep")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": base_config(args, list(wl.shapes), sorted(wl.Ms, reverse=True), MODE),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------------
def reduce_over_ranks(local_ms: float, local_units: float, dist):
    """max of the time over ranks, sum of the work: whole-job throughput of independent replicas."""
    import torch

    if dist is None:
        return local_ms, local_units
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def fp8_peak_for(peaks, timed_seconds, clocks):
    """The tensor roofline's denominator: the measured bf16 cuBLAS peak times the nominal FP8 : bf16 ratio (2).
    The burst figure when the timed region is short or the sampled clock stayed at its maximum, the sustained
    (power-capped) one for a long region whose clock dropped."""
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and
                  clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    regime = "burst" if (timed_seconds < 2.0 or at_max) else "sustained"
    return 2.0 * peaks["bf16_" + regime], regime


class Bench:
    """Device buffers of the layers and the calls into the C ABI."""

    def __init__(self, dev, rank):
        import ctypes as C

        import torch

        from paper_2307_09782_b200 import binding

        self.C, self.torch, self.binding = C, torch, binding
        self.L = binding.lib()  # fails loudly if the CUDA library is missing
        self.dev, self.rank = dev, rank
        self.stream = torch.cuda.current_stream()
        self.sp = C.c_void_p(self.stream.cuda_stream)
        self.w_cache = {}

    def vp(self, t):
        return None if t is None else self.C.c_void_p(t.data_ptr())

    def make_layer(self, wl, shape, Mmax, mode, layout, rank_lorc=RANK, copies=N_WEIGHT_COPIES):
        torch, binding = self.torch, self.binding
        K, N = shape.K, shape.N
        # replicas draw their own activations (row_offset = rank); weights are the same model on every rank
        x_bits = synth.make_x(wl.seed, Mmax, K, wl.n_outliers(K), wl.outlier_factor, row_offset=self.rank)
        x = torch.from_numpy(x_bits.view(np.int16)).to(self.dev).view(torch.bfloat16)
        key = (wl.seed, N, K, wl.sigma_w)
        if key not in self.w_cache:  # the host-side draw of a large weight takes seconds
            self.w_cache[key] = synth.make_w(wl.seed, N, K, wl.sigma_w)
        W = torch.from_numpy(self.w_cache[key]).to(self.dev)
        pw = binding.pack_weight_fp4(W, GROUP, mode, layout)
        del W
        U = V = None
        if rank_lorc:
            U_h, V_h = synth.make_lorc(wl.seed, N, K, rank_lorc)
            U, V = torch.from_numpy(U_h).to(self.dev), torch.from_numpy(V_h).to(self.dev)
        cps = [(pw.codes, pw.shift, pw.scale)]
        for _ in range(copies - 1):
            c = pw.clone()
            cps.append((c.codes, c.shift, c.scale))
        ws = binding.make_workspace(binding.linear_workspace_bytes(Mmax, N, K, rank_lorc), self.dev)
        return dict(K=K, N=N, r=rank_lorc, mode=binding.MODES[mode], layout=binding.LAYOUTS[layout], x=x, x_bits=x_bits,
                    U=U, V=V, copies=cps, ws=ws,
                    q=torch.empty((Mmax, K), dtype=torch.uint8, device=self.dev),
                    sx=torch.empty((Mmax,), dtype=torch.float32, device=self.dev),
                    t=torch.empty((Mmax, max(rank_lorc, 1)), dtype=torch.float32, device=self.dev),
                    y=torch.empty((Mmax, N), dtype=torch.float32, device=self.dev))

    def layer_call(self, ly, M, copy):
        """The whole layer through one call on raw activations."""
        vp, K, N = self.vp, ly["K"], ly["N"]
        codes, shift, scale = ly["copies"][copy % len(ly["copies"])]
        rc = self.L.zq_w4a8_linear(None, None, vp(ly["x"]), K, M, N, K, GROUP, ly["mode"], ly["layout"], vp(codes),
                                   vp(shift), vp(scale), vp(ly["U"]), vp(ly["V"]), None, ly["r"], vp(ly["y"]), 0, N,
                                   vp(ly["ws"]), ly["ws"].numel(), self.sp)
        if rc:
            raise RuntimeError(f"zq_w4a8_linear failed: {rc}")

    def quant_call(self, ly, M):
        vp, K = self.vp, ly["K"]
        rc = self.L.zq_quantize_act_fp8(vp(ly["x"]), M, K, K, vp(ly["q"]), vp(ly["sx"]), vp(ly["V"]), ly["r"],
                                        vp(ly["t"]) if ly["r"] else None, self.sp)
        if rc:
            raise RuntimeError(f"zq_quantize_act_fp8 failed: {rc}")

    def gemm_call(self, ly, M, copy):
        vp, K, N = self.vp, ly["K"], ly["N"]
        codes, shift, scale = ly["copies"][copy % len(ly["copies"])]
        rc = self.L.zq_w4a8_linear(vp(ly["q"]), vp(ly["sx"]), None, 0, M, N, K, GROUP, ly["mode"], ly["layout"],
                                   vp(codes), vp(shift), vp(scale), vp(ly["U"]), None,
                                   vp(ly["t"]) if ly["r"] else None, ly["r"], vp(ly["y"]), 0, N, vp(ly["ws"]),
                                   ly["ws"].numel(), self.sp)
        if rc:
            raise RuntimeError(f"zq_w4a8_linear failed: {rc}")

    def split_call(self, ly, M, copy, ev=None):
        """The same layer as quantizer call + GEMM call, with optional events (start, between, end)."""
        if ev:
            ev[0].record(self.stream)
        self.quant_call(ly, M)
        if ev:
            ev[1].record(self.stream)
        self.gemm_call(ly, M, copy)
        if ev:
            ev[2].record(self.stream)

    def time_shape(self, ly, M, n, batches=3):
        """Steady-state times of one (layer, M) in microseconds: the one-call layer, the quantizer alone and
        the GEMM alone on pre-quantized activations.  Each figure is one event pair around n back-to-back
        launches, divided by n (launch gaps included; an event pair around a single launch adds about 4 us of
        its own, measured with an empty kernel); the median of `batches` such batches."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn):
            res = []
            for b in range(batches + 1):  # the first batch warms up
                e0.record(self.stream)
                for i in range(n):
                    fn(b * n + i)
                e1.record(self.stream)
                torch.cuda.synchronize()
                res.append(e0.elapsed_time(e1) * 1e3 / n)
            return statistics.median(res[1:])

        t_layer = timed(lambda i: self.layer_call(ly, M, i))
        t_quant = timed(lambda i: self.quant_call(ly, M))
        t_gemm = timed(lambda i: self.gemm_call(ly, M, i))
        st = self.binding.device_status(ly["ws"])
        if st[0] != 0:
            raise RuntimeError(f"device status {st}")
        return t_layer, t_quant, t_gemm


def shape_row(name, M, N, K, r, t_layer, t_quant, t_gemm, peaks, fp8_peak, extra=None):
    row = {"layer": name, "M": M, "layer_us": round(t_layer, 2), "quant_us": round(t_quant, 2),
           "gemm_us": round(t_gemm, 2),
           "layer_tflops": round(flops(M, N, K, r) / (t_layer * 1e-6) / 1e12, 2),
           "gemm_tflops": round(2.0 * M * N * K / (t_gemm * 1e-6) / 1e12, 2),
           "weight_gbs": round(weight_bytes(N, K) / (t_gemm * 1e-6) / 1e9, 1),
           "quant_gbs": round(3.0 * M * K / (t_quant * 1e-6) / 1e9, 1),
           "gemm_frac_fp8_peak": round(2.0 * M * N * K / (t_gemm * 1e-6) / 1e12 / fp8_peak, 4),
           "gemm_frac_fp8_nominal": round(2.0 * M * N * K / (t_gemm * 1e-6) / 1e12 / NOMINAL_FP8_TFLOPS, 4),
           "gemm_frac_hbm": round(gemm_bytes(M, N, K, r) / (t_gemm * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
           "layer_frac_hbm": round(layer_bytes(M, N, K, r) / (t_layer * 1e-6) / 1e9 / peaks["hbm_gbs"], 4)}
    if extra:
        row.update(extra)
    return row


def run_ours(args):
    import torch

    from paper_2307_09782_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist_mod.init_process_group("nccl")
        dist = dist_mod
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B = Bench(dev, rank)
    binding.set_exclusive_device(not args.cooperative)  # one process, one stream of kernels per GPU

    wl = synth.WORKLOADS[WORKLOAD]
    Ms = sorted(wl.Ms, reverse=True)
    shapes = list(wl.shapes)
    mode = MODE
    sweeps = args.sweeps
    if args.case:
        parts = args.case.split(",")
        shapes = [synth.LayerShape(int(parts[0]), int(parts[1]), "case")]
        Ms = [int(parts[2])]
        if len(parts) > 3:
            mode = parts[3]
    Mmax = max(Ms)
    layers = [B.make_layer(wl, shape, Mmax, mode, args.layout) for shape in shapes]
    torch.cuda.synchronize()
    stream = B.stream
    calls = [(li, M) for M in Ms for li in range(len(layers))]
    n_big = sum(1 for _, M in calls if M == Mmax)

    def sweep(idx, events=None):
        """One pass over all (layer, M).  `events`: one triple per call at the largest token count."""
        b = 0
        for ci, (li, M) in enumerate(calls):
            copy = idx + ci // len(layers)
            if M == Mmax:
                B.split_call(layers[li], M, copy, events[b] if events else None)
                b += 1
            else:
                B.layer_call(layers[li], M, copy)

    for i in range(args.warmup):
        for s in range(sweeps):
            sweep(i * sweeps + s)
    torch.cuda.synchronize()
    for ly in layers:
        st = binding.device_status(ly["ws"])
        if st[0] != 0:
            raise RuntimeError(f"device status {st}")

    n_sw = args.steps * sweeps
    events = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_big)] for _ in range(n_sw)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = binding.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(n_sw):
        sweep(args.warmup * sweeps + i, events[i])
    e1.record(stream)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    launches = binding.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = e0.elapsed_time(e1)
    sweep_flops = sum(flops(M, layers[li]["N"], layers[li]["K"], RANK) for li, M in calls)
    ms_max, flops_all = reduce_over_ranks(total_ms, sweep_flops * n_sw, dist)
    value = flops_all / (ms_max * 1e-3) / 1e12

    # ---- dominant kernel: the GEMM at the largest token count, from the events inside the timed region
    peaks = load_peaks()
    fp8_peak, regime = fp8_peak_for(peaks, total_ms * 1e-3, clocks)
    big_layers = [li for li, M in calls if M == Mmax]
    per_layer_us = []
    for b, li in enumerate(big_layers):
        per_layer_us.append(statistics.mean(events[s][b][1].elapsed_time(events[s][b][2]) for s in range(n_sw)) * 1e3)
    bound = "tensor" if Mmax >= 512 else "hbm"
    kfam = "w4a8_mx_gemm_kernel" if args.layout == "mx" else "w4a8_gemm_kernel"
    plans = {li: binding.linear_plan(Mmax, layers[li]["N"], layers[li]["K"], mode, args.layout) for li in big_layers}
    kname = ", ".join(
        f"{'w4a8_mx_pair_gemm_kernel' if plans[li]['pair'] else kfam}<{plans[li]['bm']}> "
        f"({layers[li]['K']}->{layers[li]['N']}, {per_layer_us[b]:.1f} us)" for b, li in enumerate(big_layers))
    big_us = statistics.mean(per_layer_us)
    if bound == "tensor":
        big_flops = statistics.mean(2.0 * Mmax * layers[li]["N"] * layers[li]["K"] for li in big_layers)
        achieved = big_flops / (big_us * 1e-6) / 1e12
        roofline = {"bound": "tensor", "kernel": kname, "achieved": round(achieved, 1), "peak": round(fp8_peak, 1),
                    "unit": "TFLOP/s", "frac": round(achieved / fp8_peak, 4),
                    "peak_source": f"2 x bf16 cuBLAS peak, {regime} figure ({peaks['source']}): timed region "
                                   f"{total_ms * 1e-3:.2f} s",
                    "frac_of_burst_peak": round(achieved / (2.0 * peaks["bf16_burst"]), 4),
                    "frac_of_sustained_peak": round(achieved / (2.0 * peaks["bf16_sustained"]), 4),
                    "frac_of_nominal_4500": round(achieved / NOMINAL_FP8_TFLOPS, 4),
                    "traffic": DOMINANT_TRAFFIC if (args.layout == "mx" and not args.case) else None,
                    "launches_timed": n_sw * len(big_layers)}
    else:
        big_bytes = statistics.mean(gemm_bytes(Mmax, layers[li]["N"], layers[li]["K"], RANK) for li in big_layers)
        achieved = big_bytes / (big_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": kname, "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4),
                    "peak_source": f"copy bandwidth ({peaks['source']})", "traffic": None,
                    "launches_timed": n_sw * len(big_layers),
                    "note": "single launches between event pairs: each figure carries about 4 us of event overhead"}

    # ---- per (layer, M): steady-state times of each shape by itself, after the timed region
    table = []
    if not args.no_sweep_table:
        time.sleep(1.5)  # the timed region ends power-capped; the per-shape rows are kernels timed by themselves
        for li, M in calls:
            ly = layers[li]
            tl, tq, tg = B.time_shape(ly, M, n=20 if M <= 2048 else 6)
            table.append(shape_row(f"{ly['K']}->{ly['N']}", M, ly["N"], ly["K"], RANK, tl, tq, tg, peaks, fp8_peak))
    dec = [s for s in table if s["M"] <= 16]
    roofline_decode = None
    if dec:
        roofline_decode = {"bound": "hbm", "kernel": f"{kfam}<16>",
                           "what": "the GEMM alone on pre-quantized activations at M <= 16: algorithmic bytes / gemm_us; "
                                   "frac_whole_layer: one zq_w4a8_linear call on raw x (quantizer inside the kernel)",
                           "achieved": round(statistics.mean(s["gemm_frac_hbm"] for s in dec) * peaks["hbm_gbs"], 1),
                           "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": round(statistics.mean(s["gemm_frac_hbm"] for s in dec), 4),
                           "frac_whole_layer": round(statistics.mean(s["layer_frac_hbm"] for s in dec), 4),
                           "traffic": DECODE_TRAFFIC if (args.layout == "mx" and not args.case) else None,
                           "peak_source": f"copy bandwidth ({peaks['source']}); nominal 7700-8000"}
    big_q = [s for s in table if s["M"] == Mmax and s["layer"].startswith("28672")] or table[:1]
    roofline_quant = None
    if big_q:
        roofline_quant = {"bound": "hbm", "kernel": "activation quantizer at [%d, %s]" % (big_q[0]["M"], big_q[0]["layer"].split("->")[0]),
                          "achieved": big_q[0]["quant_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": round(big_q[0]["quant_gbs"] / peaks["hbm_gbs"], 4), "traffic": None}

    # ---- further rows the configurations ask for (not part of the timed step)
    extra_rows = []
    lorc_ms = None
    mlp_chain = None
    if not args.case and not args.no_extra:
        def extra(wl_, shape, M, md, lay, r_):
            ly = B.make_layer(wl_, shape, M, md, lay, rank_lorc=r_)
            tl, tq, tg = B.time_shape(ly, M, n=20 if M <= 2048 else 6)
            extra_rows.append(shape_row(f"{shape.K}->{shape.N}", M, shape.N, shape.K, r_, tl, tq, tg, peaks, fp8_peak,
                                        {"workload": wl_.name, "mode": md, "layout": lay, "lorc_rank": r_}))
            del ly

        other = "cast" if args.layout == "mx" else "mx"
        for shape in shapes:
            for M in (8, Mmax):  # the sweep's workload without LoRC
                extra(wl, shape, M, mode, args.layout, 0)
            for M in (1, 8, Mmax):  # the other kernel family (cast: kind::f8f6f4, E4M3 x E4M3, the kernel casts)
                extra(wl, shape, M, mode, other, RANK)
        for shape in shapes:  # FP8-E4M3 weights (W8A8 FP - FP) through the block-scaled kernel
            for M in (8, Mmax):
                extra(wl, shape, M, mode, "mx_fp8", RANK)
        extra(wl, shapes[0], Mmax, mode, "cast_e5m2", RANK)  # E5M2 as the cast target
        # LoRC factor construction on the device (offline step), rank 8, two power iterations
        shape = shapes[0]
        Wd = torch.from_numpy(B.w_cache[(wl.seed, shape.N, shape.K, wl.sigma_w)]).to(dev)
        pw = binding.pack_weight_fp4(Wd, GROUP, mode, "mx")
        om = torch.randn((shape.K, RANK + 8), dtype=torch.float32, device=dev)
        binding.lorc_factors(Wd, pw, RANK, om, iters=2)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        binding.lorc_factors(Wd, pw, RANK, om, iters=2)
        torch.cuda.synchronize()
        lorc_ms = (time.perf_counter() - t0) * 1e3
        del Wd, pw, om
        # the quantizer when the layer before has collected the tokens' maxima in its epilogue
        # (zq_w4a8_linear_fused_out -> zq_quantize_act_fp8_scaled): one pass, at the largest activation of the sweep
        qshape = max(shapes, key=lambda sh: sh.K)
        ly = B.make_layer(wl, qshape, Mmax, mode, args.layout)
        amax = torch.cat([ly["x"][i:i + 512].float().abs().amax(dim=1) for i in range(0, Mmax, 512)]).contiguous()
        vp_ = B.vp

        def scaled_call():
            rc = B.L.zq_quantize_act_fp8_scaled(vp_(ly["x"]), Mmax, qshape.K, qshape.K, vp_(amax), vp_(ly["q"]),
                                                vp_(ly["sx"]), vp_(ly["V"]), ly["r"],
                                                vp_(ly["t"]) if ly["r"] else None, B.sp)
            if rc:
                raise RuntimeError(f"zq_quantize_act_fp8_scaled failed: {rc}")
        res = []
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for b in range(4):
            ev0.record(B.stream)
            for _ in range(6):
                scaled_call()
            ev1.record(B.stream)
            torch.cuda.synchronize()
            res.append(ev0.elapsed_time(ev1) * 1e3 / 6)
        us1 = statistics.median(res[1:])
        if roofline_quant is not None:
            gbs1 = 3.0 * Mmax * qshape.K / (us1 * 1e-6) / 1e9
            roofline_quant["one_pass_given_maxima"] = {
                "what": "zq_quantize_act_fp8_scaled at the same shape: the token maxima come from the epilogue of the "
                        "layer before (zq_w4a8_linear_fused_out), so x is read once and nothing is reduced",
                "us": round(us1, 2), "achieved": round(gbs1, 1), "frac": round(gbs1 / peaks["hbm_gbs"], 4)}
        del ly, amax
        # The two layers chained as an MLP block at the largest token count, fc1 -> ReLU -> fc2, with and without
        # the fusion on the output side: fused = fc1 with ReLU and the token maxima in its epilogue (bf16 y), the
        # one-pass quantizer, fc2; unfused = fc1 (bf16 y), a separate ReLU pass, the two-pass quantizer, fc2.
        if len(shapes) == 2 and shapes[0].N == shapes[1].K:
            l1 = B.make_layer(wl, shapes[0], Mmax, mode, args.layout, copies=1)
            l2 = B.make_layer(wl, shapes[1], Mmax, mode, args.layout, copies=1)
            y1 = torch.empty((Mmax, shapes[0].N), dtype=torch.bfloat16, device=dev)
            am1 = torch.empty((Mmax,), dtype=torch.float32, device=dev)
            vp_ = B.vp

            def fc(ly, x_raw, q_, sx_, t_, y_, ydt, relu, amax_):
                c_, sh_, sc_ = ly["copies"][0]
                args_ = (vp_(q_), vp_(sx_), vp_(x_raw), ly["K"], Mmax, ly["N"], ly["K"], GROUP, ly["mode"], ly["layout"],
                         vp_(c_), vp_(sh_), vp_(sc_), vp_(ly["U"]), vp_(ly["V"]) if x_raw is not None else None,
                         vp_(t_) if (t_ is not None and ly["r"]) else None, ly["r"], vp_(y_), ydt, ly["N"], vp_(ly["ws"]),
                         ly["ws"].numel(), B.sp)
                rc = (B.L.zq_w4a8_linear_fused_out(*args_, 1 if relu else 0, vp_(amax_)) if (relu or amax_ is not None)
                      else B.L.zq_w4a8_linear(*args_))
                if rc:
                    raise RuntimeError(f"linear failed in the MLP chain: {rc}")

            def quant2(scaled):
                a_ = (vp_(y1), Mmax, l2["K"], l2["K"])
                b_ = (vp_(l2["q"]), vp_(l2["sx"]), vp_(l2["V"]), l2["r"], vp_(l2["t"]) if l2["r"] else None, B.sp)
                rc = (B.L.zq_quantize_act_fp8_scaled(*a_, vp_(am1), *b_) if scaled else B.L.zq_quantize_act_fp8(*a_, *b_))
                if rc:
                    raise RuntimeError(f"quantizer failed in the MLP chain: {rc}")

            def fused():
                fc(l1, l1["x"], None, None, None, y1, 1, True, am1)
                quant2(True)
                fc(l2, None, l2["q"], l2["sx"], l2["t"], l2["y"], 0, False, None)

            def fused_relu():
                fc(l1, l1["x"], None, None, None, y1, 1, True, None)
                quant2(False)
                fc(l2, None, l2["q"], l2["sx"], l2["t"], l2["y"], 0, False, None)

            def unfused():
                fc(l1, l1["x"], None, None, None, y1, 1, False, None)
                torch.relu_(y1)
                quant2(False)
                fc(l2, None, l2["q"], l2["sx"], l2["t"], l2["y"], 0, False, None)

            def timed3(fn, n=4):
                res = []
                e0_, e1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                for b in range(3):
                    e0_.record(B.stream)
                    for _ in range(n):
                        fn()
                    e1_.record(B.stream)
                    torch.cuda.synchronize()
                    res.append(e0_.elapsed_time(e1_) * 1e3 / n)
                return statistics.median(res[1:])
            # interleaved, so that all three see the same clocks
            runs_ = {"u": [], "r": [], "f": []}
            for rep_ in range(3):
                for key_, fn_ in (("u", unfused), ("r", fused_relu), ("f", fused)):
                    runs_[key_].append(timed3(fn_, n=2))
            tu_, tr_, tf_ = (statistics.median(runs_[k_]) for k_ in ("u", "r", "f"))
            fl_ = flops(Mmax, shapes[0].N, shapes[0].K, RANK) + flops(Mmax, shapes[1].N, shapes[1].K, RANK)
            mlp_chain = {"what": "fc1 -> ReLU -> fc2 at M = %d, bf16 between the layers, FP32 out: separate ReLU pass; "
                                 "ReLU in fc1's epilogue; ReLU and the token maxima in fc1's epilogue with the "
                                 "one-pass quantizer" % Mmax,
                         "unfused_us": round(tu_, 1), "relu_fused_us": round(tr_, 1), "relu_and_maxima_fused_us": round(tf_, 1),
                         "unfused_tflops": round(fl_ / (tu_ * 1e-6) / 1e12, 1),
                         "relu_fused_tflops": round(fl_ / (tr_ * 1e-6) / 1e12, 1),
                         "relu_and_maxima_fused_tflops": round(fl_ / (tf_ * 1e-6) / 1e12, 1)}
            del l1, l2, y1, am1
        wl7 = synth.WORKLOADS["llama7b"]  # unconstrained scales (per-group FP32 promotion) at 2048 tokens
        for shape in wl7.shapes:
            for md, lay in EXTRA_LLAMA7B:
                extra(wl7, shape, 2048, md, lay, RANK)
        torch.cuda.empty_cache()

    # ---- end to end through the host-buffer entry point (host <-> device copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        import ctypes as C

        h2d = d2h = 0
        hosts = []
        for ly in layers:
            K, N = ly["K"], ly["N"]
            xh = torch.from_numpy(ly["x_bits"].view(np.int16)).view(torch.bfloat16).pin_memory()
            yh = torch.empty((Mmax, N), dtype=torch.float32).pin_memory()
            wsh = binding.make_workspace(binding.linear_host_workspace_bytes(Mmax, N, K, RANK), dev)
            hosts.append((xh, yh, wsh))

        def e2e_sweep(idx):
            for ci, (li, M) in enumerate(calls):
                ly = layers[li]
                xh, yh, wsh = hosts[li]
                codes, shift, scale = ly["copies"][(idx + ci // len(layers)) % N_WEIGHT_COPIES]
                rc = B.L.zq_w4a8_linear_host(C.c_void_p(xh.data_ptr()), M, ly["N"], ly["K"], GROUP, ly["mode"],
                                             ly["layout"], B.vp(codes), B.vp(shift), B.vp(scale), B.vp(ly["U"]),
                                             B.vp(ly["V"]), RANK, C.c_void_p(yh.data_ptr()), B.vp(wsh), wsh.numel(), B.sp)
                if rc:
                    raise RuntimeError(f"zq_w4a8_linear_host failed: {rc}")

        for li, M in calls:
            h2d += 2 * M * layers[li]["K"]
            d2h += 4 * M * layers[li]["N"]
        e2e_sweeps = max(1, min(args.steps, 5))
        e2e_sweep(0)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_sweeps):
            e2e_sweep(i + 1)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
        if dist:
            dist.barrier()
        e2e_ms_max, e2e_flops = reduce_over_ranks(e2e_ms, sweep_flops * e2e_sweeps, dist)
        e2e = {"value": round(e2e_flops / (e2e_ms_max * 1e-3) / 1e12, 3), "unit": UNIT,
               "h2d_bytes_per_step": h2d * sweeps, "d2h_bytes_per_step": d2h * sweeps,
               "sweeps_timed": e2e_sweeps, "ms_per_sweep": round(e2e_ms_max / e2e_sweeps, 3),
               "api": "zq_w4a8_linear_host (pinned host x -> device, quantizer + linear, y -> pinned host)"}

    if rank != 0:
        return
    cfg = base_config(args, shapes, Ms, mode)
    cfg.update({"sweeps_per_step": sweeps, "multi_gpu": "independent replicas",
                "l2": f"inputs larger than L2: {N_WEIGHT_COPIES} weight copies per layer rotated, >300 MB "
                      "streamed between two reads of one buffer"})
    dtype = ("f4e2m1 (E8M0 block scale) x f8e4m3 -> f32" if args.layout == "mx"
             else "f8e4m3 (cast from f4e2m1 in the kernel) x f8e4m3 -> f32")
    line = {"metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_max / args.steps, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic", "config": cfg,
            "timed_region_s": round(ms_max * 1e-3, 3),
            "roofline": roofline, "roofline_decode": roofline_decode, "roofline_quant": roofline_quant,
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "sweep_note": "per-shape rows: each (layer, M) timed by itself after the timed region and a 1.5 s pause: one event pair "
                          "around n = 6-20 back-to-back launches (rotated weight copies), divided by n, median of 3 "
                          "batches; layer_us = one zq_w4a8_linear call on raw x; quant_us / gemm_us = the quantizer "
                          "kernel alone and the GEMM alone on pre-quantized activations; the table is taken at the clocks "
                          "the power cap leaves after the timed region (in a fresh process the shapes up to 2048 tokens "
                          "read 1.2-1.6 x faster, e.g. the GEMMs at 512 tokens 93 us)",
            "sweep": table, "extra_rows": extra_rows, "lorc_factors_ms": lorc_ms, "mlp_chain": mlp_chain}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(wl)
    print(json.dumps(line))


def spawn_ranks(args) -> int:
    """`--gpus N` without a torchrun environment: start the N ranks (one process per GPU) ourselves."""
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--sweeps", type=int, default=25,
                    help="passes over the (layer, M) sweep per step (a step of about 0.1 s, so that 20 steps give "
                         "a timed region of about 2 s and settled clocks)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the rows outside the timed step")
    ap.add_argument("--no-sweep-table", action="store_true", help="skip the per-shape table")
    ap.add_argument("--cooperative", action="store_true",
                    help="keep the library's default cooperative launches (the bench has the device to itself and "
                         "says so to the library, which then launches plainly: about 3.5 us less per shared-tile launch)")
    ap.add_argument("--layout", default="mx", choices=["cast", "mx"],
                    help="weight layout: the kernel casts FP4 to FP8 (cast) or the tensor core does (mx)")
    ap.add_argument("--case", default=None, metavar="K,N,M[,MODE]",
                    help="time one layer shape at one token count instead of the sweep (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    run_ours(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
