"""Benchmark of the W4A8 quantized linear layer (FP4 weights, FP8 activations, LoRC) on B200.

A step is one pass of the whole hot path (token-wise FP8 quantization with the LoRC down-projection,
then the W4A8 GEMM with its scale + LoRC epilogue) over the OPT-30B-shaped sweep: the two MLP layers
(7168 -> 28672 and 28672 -> 7168), each at M in {1, 8, 32, 128, 512, 2048, 8192} tokens, constraint M2,
group 128, LoRC rank 8.  Weights are packed once before the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-cpu-baseline]

Prints one JSON line.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
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
# ncu, one pass, the bench's own M = 8192 launches of w4a8_mx_gemm_kernel<224> / <256> (profiles/): 1510.6 MB and 1655.4 MB
DOMINANT_TRAFFIC = 1583.0e6
# ncu --set full, w4a8_mx_gemm_kernel<16> at 7168->28672, M = 8 (profiles/): read + write of the two captured launches
DECODE_TRAFFIC = 114.6e6
METRIC = "w4a8_linear_tflops"
UNIT = "TFLOP/s"
N_WEIGHT_COPIES = 2  # per layer; rotated so that > 2x the L2 size streams between two reads of one buffer


def flops(M, N, K, r):
    return 2.0 * M * N * K + 2.0 * M * r * (K + N)


def algorithmic_bytes(M, N, K, r, group=GROUP):
    """Bytes the fused path must move (M1/M2, FP32 y): codes, shifts, channel scales, x, y, U, V."""
    return N * K / 2 + N * K / group + 4 * N + 2 * M * K + 4 * M * N + 2 * r * (N + K)


def weight_bytes(N, K, group=GROUP):
    return N * K / 2 + N * K / group + 4 * N


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
            "config": {"workload": WORKLOAD, "group": GROUP, "mode": MODE, "lorc_rank": RANK},
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
    binding.lib()  # fails loudly if the CUDA library is missing

    wl = synth.WORKLOADS[WORKLOAD]
    Ms = list(wl.Ms)
    shapes = list(wl.shapes)
    mode = MODE
    layout = binding.LAYOUTS[args.layout]
    if args.case:
        parts = args.case.split(",")
        shapes = [synth.LayerShape(int(parts[0]), int(parts[1]), "case")]
        Ms = [int(parts[2])]
        if len(parts) > 3:
            mode = parts[3]
    Mmax = max(Ms)
    layers = []
    for shape in shapes:
        K, N = shape.K, shape.N
        # replicas draw their own activations (row_offset = rank); weights are the same model on every rank
        x_bits = synth.make_x(wl.seed, Mmax, K, wl.n_outliers(K), wl.outlier_factor, row_offset=rank)
        x = torch.from_numpy(x_bits.view(np.int16)).to(dev).view(torch.bfloat16)
        W = torch.from_numpy(synth.make_w(wl.seed, N, K, wl.sigma_w)).to(dev)
        pw = binding.pack_weight_fp4(W, GROUP, mode, layout)
        del W
        U_h, V_h = synth.make_lorc(wl.seed, N, K, RANK)
        U, V = torch.from_numpy(U_h).to(dev), torch.from_numpy(V_h).to(dev)
        copies = [(pw.codes, pw.shift, pw.scale)]
        for _ in range(N_WEIGHT_COPIES - 1):
            c = pw.clone()
            copies.append((c.codes, c.shift, c.scale))
        ws = binding.make_workspace(binding.linear_workspace_bytes(Mmax, N, K, RANK), dev)
        layers.append(dict(K=K, N=N, x=x, x_bits=x_bits, U=U, V=V, copies=copies, ws=ws,
                           q=torch.empty((Mmax, K), dtype=torch.uint8, device=dev),
                           sx=torch.empty((Mmax,), dtype=torch.float32, device=dev),
                           t=torch.empty((Mmax, RANK), dtype=torch.float32, device=dev),
                           y=torch.empty((Mmax, N), dtype=torch.float32, device=dev)))
    torch.cuda.synchronize()

    L = binding.lib()
    import ctypes as C

    def vp(t):
        return None if t is None else C.c_void_p(t.data_ptr())

    stream = torch.cuda.current_stream()
    sp = C.c_void_p(stream.cuda_stream)
    calls = [(li, M) for M in Ms for li in range(len(layers))]

    def one_call(li, M, copy, ev=None):
        ly = layers[li]
        K, N = ly["K"], ly["N"]
        codes, shift, scale = ly["copies"][copy]
        if ev:
            ev[0].record(stream)
        rc = L.zq_quantize_act_fp8(vp(ly["x"]), M, K, K, vp(ly["q"]), vp(ly["sx"]), vp(ly["V"]), RANK, vp(ly["t"]), sp)
        if ev:
            ev[1].record(stream)
        rc |= L.zq_w4a8_linear(vp(ly["q"]), vp(ly["sx"]), None, 0, M, N, K, GROUP, binding.MODES[mode], layout, vp(codes),
                               vp(shift), vp(scale), vp(ly["U"]), None, vp(ly["t"]), RANK, vp(ly["y"]), 0, N,
                               vp(ly["ws"]), ly["ws"].numel(), sp)
        if ev:
            ev[2].record(stream)
        if rc:
            raise RuntimeError(f"zqfp call failed: {rc}")

    def step(idx, events=None):
        for ci, (li, M) in enumerate(calls):
            one_call(li, M, (idx + ci // len(layers)) % N_WEIGHT_COPIES, events[ci] if events else None)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    for ly in layers:
        st = binding.device_status(ly["ws"])
        if st[0] != 0:
            raise RuntimeError(f"device status {st}")

    events = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in calls] for _ in range(args.steps)]
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
    for i in range(args.steps):
        step(args.warmup + i, events[i])
    e1.record(stream)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    launches = binding.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = e0.elapsed_time(e1)
    step_flops = sum(flops(M, layers[li]["N"], layers[li]["K"], RANK) for li, M in calls)
    ms_max, flops_all = reduce_over_ranks(total_ms, step_flops * args.steps, dist)
    value = flops_all / (ms_max * 1e-3) / 1e12

    # ---- per-call table from the events of the timed region
    peaks = load_peaks()
    fp8_peak = 2.0 * peaks["bf16_sustained"]
    sweep = []
    for ci, (li, M) in enumerate(calls):
        ly = layers[li]
        K, N = ly["K"], ly["N"]
        tq = statistics.mean(events[s][ci][0].elapsed_time(events[s][ci][1]) for s in range(args.steps)) * 1e3
        tg = statistics.mean(events[s][ci][1].elapsed_time(events[s][ci][2]) for s in range(args.steps)) * 1e3
        gemm_bytes = weight_bytes(N, K) + M * K + 4 * M + 4 * M * N + 2 * RANK * N + 4 * M * RANK
        sweep.append({"layer": f"{K}->{N}", "M": M, "quant_us": round(tq, 2), "gemm_us": round(tg, 2),
                      "gemm_tflops": round(2.0 * M * N * K / (tg * 1e-6) / 1e12, 2),
                      "weight_gbs": round(weight_bytes(N, K) / (tg * 1e-6) / 1e9, 1),
                      "gemm_gbs": round(gemm_bytes / (tg * 1e-6) / 1e9, 1),
                      "quant_gbs": round(3.0 * M * K / (tq * 1e-6) / 1e9, 1),
                      "frac_fp8_peak": round(2.0 * M * N * K / (tg * 1e-6) / 1e12 / fp8_peak, 4),
                      "frac_hbm": round(gemm_bytes / (tg * 1e-6) / 1e9 / peaks["hbm_gbs"], 4)})
    # dominant kernel: the GEMM at the largest M (both layers)
    big = [s for s in sweep if s["M"] == Mmax]
    big_flops = sum(2.0 * Mmax * ly["N"] * ly["K"] for ly in layers) / len(layers)
    big_us = statistics.mean(s["gemm_us"] for s in big)
    achieved = big_flops / (big_us * 1e-6) / 1e12
    roofline = {"bound": "tensor", "kernel": "w4a8_mx_gemm_kernel<224> (7168->28672), <256> (28672->7168)" if layout else "w4a8_gemm_kernel<256,false>", "achieved": round(achieved, 1),
                "peak": round(fp8_peak, 1), "unit": "TFLOP/s", "frac": round(achieved / fp8_peak, 4),
                "traffic": DOMINANT_TRAFFIC if (layout and not args.case) else None,
                "traffic_note": "DRAM bytes per launch (ncu dram__bytes_read + write, mean of the two M = 8192 launches)",
                "peak_source": f"2 x bf16 sustained cuBLAS peak ({peaks['source']}); nominal dense FP8 4500"}
    dec = [s for s in sweep if s["M"] <= 16] or [sweep[0]]
    roofline_decode = {"bound": "hbm", "kernel": "w4a8_mx_gemm_kernel<16>" if layout else "w4a8_gemm_kernel<16,false>",
                       "achieved": round(statistics.mean(s["gemm_gbs"] for s in dec), 1),
                       "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": round(statistics.mean(s["frac_hbm"] for s in dec), 4),
                       "traffic": DECODE_TRAFFIC if (layout and not args.case) else None,
                       "traffic_note": "DRAM bytes per launch (ncu, 7168->28672 at M = 8, mean of two launches)",
                       "peak_source": f"copy bandwidth ({peaks['source']}); nominal 7700-8000"}
    big_q = [s for s in sweep if s["M"] == Mmax and s["layer"].startswith("28672")] or [sweep[-1]]
    roofline_quant = {"bound": "hbm", "kernel": "act_quant_rows_kernel<true>", "achieved": big_q[0]["quant_gbs"],
                      "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(big_q[0]["quant_gbs"] / peaks["hbm_gbs"], 4),
                      "traffic": None}

    # ---- end to end through the host-buffer entry point (host <-> device copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        h2d = d2h = 0
        hosts = []
        for ly in layers:
            K, N = ly["K"], ly["N"]
            xh = torch.from_numpy(ly["x_bits"].view(np.int16)).view(torch.bfloat16).pin_memory()
            yh = torch.empty((Mmax, N), dtype=torch.float32).pin_memory()
            wsh = binding.make_workspace(binding.linear_host_workspace_bytes(Mmax, N, K, RANK), dev)
            hosts.append((xh, yh, wsh))

        def e2e_step(idx):
            for ci, (li, M) in enumerate(calls):
                ly = layers[li]
                xh, yh, wsh = hosts[li]
                codes, shift, scale = ly["copies"][(idx + ci // len(layers)) % N_WEIGHT_COPIES]
                rc = L.zq_w4a8_linear_host(C.c_void_p(xh.data_ptr()), M, ly["N"], ly["K"], GROUP, binding.MODES[mode], layout,
                                           vp(codes), vp(shift), vp(scale), vp(ly["U"]), vp(ly["V"]), RANK,
                                           C.c_void_p(yh.data_ptr()), vp(wsh), wsh.numel(), sp)
                if rc:
                    raise RuntimeError(f"zq_w4a8_linear_host failed: {rc}")

        for li, M in calls:
            h2d += 2 * M * layers[li]["K"]
            d2h += 4 * M * layers[li]["N"]
        e2e_steps = max(1, min(args.steps, 5))
        e2e_step(0)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            e2e_step(i + 1)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
        if dist:
            dist.barrier()
        e2e_ms_max, e2e_flops = reduce_over_ranks(e2e_ms, step_flops * e2e_steps, dist)
        e2e = {"value": round(e2e_flops / (e2e_ms_max * 1e-3) / 1e12, 3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": round(e2e_ms_max / e2e_steps, 3),
               "api": "zq_w4a8_linear_host (pinned host x -> device, quantizer + linear, y -> pinned host)"}

    if rank != 0:
        return
    line = {"metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_max / args.steps, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f8e4m3 x f8e4m3 -> f32", "data": "synthetic",
            "config": {"workload": WORKLOAD if not args.case else f"case {args.case}",
                       "layers": [f"{s.K}->{s.N}" for s in shapes], "M": Ms, "group": GROUP, "mode": mode, "weight_layout": args.layout, "lorc_rank": RANK, "multi_gpu": "independent replicas",
                       "l2": f"inputs larger than L2: {N_WEIGHT_COPIES} weight copies per layer rotated, >300 MB "
                             "streamed between two reads of one buffer"},
            "roofline": roofline, "roofline_decode": roofline_decode, "roofline_quant": roofline_quant,
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "sweep": sweep}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(wl)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layout", default="mx", choices=["cast", "mx"],
                    help="weight layout: the kernel casts FP4 to FP8 (cast) or the tensor core does (mx)")
    ap.add_argument("--case", default=None, metavar="K,N,M[,MODE]",
                    help="time one layer shape at one token count instead of the sweep (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
