#!/usr/bin/env python
"""Benchmark of the SmoothRot W4A4 linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1|cfg2|cfg3]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

One "step" is one pass of the whole path over one batch of seeded synthetic
input: calibrate (per-channel absmax -> scales), fuse_weights (scale, rotate,
quantize, pack W), quant_act (Hadamard + per-token INT4 quantize + pack X) and
linear (INT4 x INT4 GEMM + dequant to fp16).  The headline value is the layer's
2*M*N*K integer operations divided by the time of the whole step.

The device-timed region keeps every input resident in HBM; between steps the
loop rotates through several distinct buffer sets whose total size exceeds
twice the L2 capacity, so no step finds its inputs in L2.  A step is launched
as two CUDA graphs recorded from the library calls, so that the Python cost of
a launch (longer than some of the kernels) does not sit in the device timeline;
a pair of events around the second graph times the GEMM kernel inside the
timed region.  The end-to-end figure starts from pinned host buffers, makes the
calls eagerly and ends with the output back on the host, with the copies
inside the timed region.

Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_05413_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
# DRAM bytes (read + write) of one launch of the GEMM kernel from an ncu capture, by (M, N, K);
# absent (None in the output) for shapes that were not captured or after the kernel changed.
LINEAR_TRAFFIC = {(2048, 6144, 4096): 16.85e6 + 0.04e6}   # operands from DRAM; Y (25.2 MB) still in L2 at kernel end
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
METRIC = "w4a4_smoothrot_linear_tops"
UNIT = "TOPS"

WORKLOADS = {
    "cfg0": (synth.config0, "configs[0]: tiny layer, X [64 x 128], W [256 x 128]"),
    "cfg1": (synth.config1, "configs[1]: LLaMA-3.1-8B-shaped fused QKV, X [2048 x 4096], W [6144 x 4096]"),
    "cfg2": (synth.config2, "configs[2]: down_proj with online Hadamard, X [2048 x 14336], W [4096 x 14336]"),
    "cfg3": (synth.config3, "configs[3]: fused gate/up, X [8192 x 4096], W [28672 x 4096]"),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TFLOPS, bf16_sustained=1400.0, source="fallback")


def layer_ops(M, N, K):
    return 2.0 * M * N * K


def algorithmic_bytes(M, N, K, T):
    """Bytes each call must move at least once (fp16 in, packed codes out, fp32 scales)."""
    return {
        "calibrate": 2.0 * T * K + 2.0 * N * K + 4.0 * K * 5,
        "fuse_weights": 2.0 * N * K + 0.5 * N * K + 4.0 * N + 4.0 * K,
        "quant_act": 2.0 * M * K + 0.5 * M * K + 4.0 * M + 4.0 * K,
        "linear": 0.5 * M * K + 0.5 * N * K + 2.0 * M * N + 4.0 * (M + N),
    }


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
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
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, flag in zip(names, parts[4:8]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)),
                "power_w_max": float(max(power)), "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------
# The CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# ---------------------------------------------------------------------------
def oracle_step(case, Ms, Ns):
    """One pass of the whole path by the oracle on the first Ms tokens and Ns
    output channels of the workload (full K, full calibration set); returns seconds."""
    from oracle import smoothrot_oracle as orc
    t0 = time.perf_counter()
    orc.smoothrot_layer(case.X[:Ms], case.X_calib, case.W[:Ns], case.d, case.alpha, case.clip_a, case.clip_w)
    return time.perf_counter() - t0


def oracle_sample_shape(case):
    """A bounded sample of the workload: the whole layer if its GEMM has at most
    6e10 multiply-adds (a few seconds for the plain C loop), else the leading
    tokens / output channels, halved in turn until it does."""
    Ms, Ns = case.M, case.N
    while float(Ms) * Ns * case.K > 6e10:
        if Ms >= Ns and Ms > 1:
            Ms //= 2
        else:
            Ns = max(8, Ns // 2)
    return Ms, Ns


def oracle_threads():
    from oracle import smoothrot_oracle as orc
    return orc.gemm_threads()


def run_reference(args, case, desc):
    Ms, Ns = oracle_sample_shape(case)
    for _ in range(min(args.warmup, 1)):
        oracle_step(case, Ms, Ns)
    steps = max(1, min(args.steps, 3))
    t = [oracle_step(case, Ms, Ns) for _ in range(steps)]
    sec = float(np.mean(t))
    value = layer_ops(Ms, Ns, case.K) / sec / 1e12
    sample = f"first {Ms} tokens x first {Ns} output channels, full K = {case.K}, whole path per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int4", "data": "synthetic",
        "config": {"workload": desc, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# The GPU arm
# ---------------------------------------------------------------------------
class DeviceSet:
    """One resident copy of a layer's inputs and outputs."""

    def __init__(self, torch, sr, case, dev):
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        M, N, K = case.M, case.N, case.K
        self.X, self.Xc, self.W, self.d = t(case.X), t(case.X_calib), t(case.W), t(case.d)
        f32 = lambda n: torch.empty(n, dtype=torch.float32, device=dev)
        self.amax, self.s, self.pre_w, self.pre_x = f32(K), f32(K), f32(K), f32(K)
        self.wq = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
        self.xq = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
        self.dw, self.dx = f32(N), f32(M)
        self.Y = torch.empty((M, N), dtype=torch.float16, device=dev)
        need = sr.workspace_bytes(M, N, K)
        self.ws = torch.empty(need, dtype=torch.uint8, device=dev) if need else None

    def nbytes(self):
        tensors = (self.X, self.Xc, self.W, self.wq, self.xq, self.Y)
        return sum(x.numel() * x.element_size() for x in tensors)


CALLS = ("calibrate", "fuse_weights", "quant_act", "linear")


def step_calls(sr, case, ds):
    """The four calls of the path on one buffer set, in order, as closures."""
    def calibrate():
        ds.amax.zero_()
        sr.calibrate(ds.Xc, ds.amax, W=ds.W, alpha=case.alpha, s_out=ds.s, d=ds.d,
                     pre_w_out=ds.pre_w, pre_x_out=ds.pre_x)
    return {
        "calibrate": calibrate,
        "fuse_weights": lambda: sr.fuse_weights(ds.W, ds.pre_w, case.clip_w, ds.wq, ds.dw),
        "quant_act": lambda: sr.quant_act(ds.X, ds.pre_x, case.clip_a, ds.xq, ds.dx),
        "linear": lambda: sr.linear(ds.xq, ds.dx, ds.wq, ds.dw, ds.Y, ds.ws),
    }


def gpu_step(sr, case, ds):
    """The whole path on one buffer set, call by call (eager launches)."""
    for fn in step_calls(sr, case, ds).values():
        fn()


def max_over_ranks(torch, dist, value, dev):
    """The slowest rank's figure (a time): what a multi-GPU number is quoted on.  `dist` is
    torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def capture(torch, fns):
    """Records the given calls (made through the binding, on the capturing stream) into one CUDA graph."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for fn in fns:
            fn()
    return g


def run_gpu(args, case, desc):
    import torch
    from paper_2506_05413_b200 import binding as sr

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    sr.load()
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    M, N, K, T = case.M, case.N, case.K, case.X_calib.shape[0]
    first = DeviceSet(torch, sr, case, dev)
    n_sets = max(2, int(np.ceil(2.2 * L2_BYTES / first.nbytes())))
    sets = [first]
    for i in range(1, n_sets):
        ds = DeviceSet(torch, sr, case, dev)
        sets.append(ds)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for i in range(warmup):
        gpu_step(sr, case, sets[i % n_sets])
    torch.cuda.synchronize()
    assert sr.device_status() == 0, "a device-side wait timed out during warm-up"

    # A step is replayed as two CUDA graphs per buffer set, recorded from the same C-ABI calls:
    # [calibrate, fuse_weights, quant_act] and [linear].  The split lets a pair of events bracket
    # the dominant kernel inside the timed region; the Python launch cost of eager calls (longer
    # than some of the kernels) stays out of the device timeline.
    launches0 = sr.launch_count()
    front, back, single = [], [], {name: [] for name in CALLS}
    for ds in sets:
        calls = step_calls(sr, case, ds)
        front.append(capture(torch, [calls["calibrate"], calls["fuse_weights"], calls["quant_act"]]))
        back.append(capture(torch, [calls["linear"]]))
    launches_per_step = (sr.launch_count() - launches0) // n_sets
    for ds in sets:
        calls = step_calls(sr, case, ds)
        for name in CALLS:
            single[name].append(capture(torch, [calls[name]]))
    for i in range(warmup):
        front[i % n_sets].replay()
        back[i % n_sets].replay()
    torch.cuda.synchronize()

    # ---- device-timed region: K steps ------------------------------------------------
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    start.record()
    for i in range(args.steps):
        front[i % n_sets].replay()
        ev[i][0].record()
        back[i % n_sets].replay()
        ev[i][1].record()
    stop.record()
    barrier()
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(torch, dist, start.elapsed_time(stop), dev)
    ms_per_step = total_ms / args.steps
    linear_live_ms = float(np.mean([ev[i][0].elapsed_time(ev[i][1]) for i in range(args.steps)]))
    assert sr.device_status() == 0, "a device-side wait timed out"

    # ---- each call alone (outside the timed region): one graph per call and buffer set ----
    call_ms = {}
    reps = max(10, min(args.steps, 100))
    for name in CALLS:
        gs = single[name]
        for i in range(3):
            gs[i % n_sets].replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(reps):
            gs[i % n_sets].replay()
        e1.record()
        torch.cuda.synchronize()
        call_ms[name] = e0.elapsed_time(e1) / reps
    call_ms_alone_linear = call_ms["linear"]
    call_ms["linear"] = linear_live_ms

    # ---- end to end: pinned host inputs -> device -> path -> output on the host ----
    # Every step copies its own inputs from pinned host memory and reads its own output back.  The
    # steps rotate through the buffer sets on three streams (copy in, compute, copy out), ordered by
    # events, so that the two PCIe directions and the kernels of neighbouring steps overlap, as a
    # serving loop would run them; the clock stops when the last output has reached the host.
    host_in = [torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in (case.X, case.X_calib, case.W, case.d)]
    host_Y = [torch.empty((M, N), dtype=torch.float16).pin_memory() for _ in sets]
    h2d = sum(h.numel() * h.element_size() for h in host_in)
    d2h = host_Y[0].numel() * host_Y[0].element_size()
    s_in, s_run, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
    ev_in = [torch.cuda.Event() for _ in sets]
    ev_run = [torch.cuda.Event() for _ in sets]
    ev_out = [torch.cuda.Event() for _ in sets]

    def e2e_steps_run(count):
        torch.cuda.synchronize()
        for i in range(count):
            k = i % len(sets)
            ds = sets[k]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_run[k])          # the set's inputs are no longer being read
                for h, d_ in zip(host_in, (ds.X, ds.Xc, ds.W, ds.d)):
                    d_.copy_(h, non_blocking=True)
                ev_in[k].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[k])
                s_run.wait_event(ev_out[k])         # the set's previous output has left the device
                gpu_step(sr, case, ds)
                ev_run[k].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[k])
                host_Y[k].copy_(ds.Y, non_blocking=True)
                ev_out[k].record(s_out)
        torch.cuda.synchronize()

    e2e_steps_run(3)
    e2e_steps = max(3, min(args.steps, 20))
    barrier()
    t0 = time.perf_counter()
    e2e_steps_run(e2e_steps)
    barrier()
    e2e_sec = max_over_ranks(torch, dist, (time.perf_counter() - t0) / e2e_steps, dev)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ops = layer_ops(M, N, K)
    peaks = measured_peaks()
    int8_peak = peaks["bf16"] * (NOMINAL_INT8_TOPS / NOMINAL_BF16_TFLOPS)
    abytes = algorithmic_bytes(M, N, K, T)
    dominant = max(call_ms, key=call_ms.get)
    if dominant == "linear":
        achieved = ops / (call_ms["linear"] * 1e-3) / 1e12
        roofline = {"kernel": "w4a4_gemm_pair_tmem_kernel (smoothrot_linear)", "bound": "tensor", "achieved": achieved,
                    "peak": int8_peak, "unit": "TOP/s", "frac": achieved / int8_peak, "traffic": LINEAR_TRAFFIC.get((M, N, K)),
                    "timed": "CUDA events around the kernel's launch inside the timed region, mean over the steps",
                    "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16']} TFLOP/s x 2 (nominal int8:bf16 ratio)",
                    "frac_of_nominal_4500": achieved / NOMINAL_INT8_TOPS}
    else:
        achieved = abytes[dominant] / (call_ms[dominant] * 1e-3) / 1e9
        roofline = {"kernel": dominant, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                    "timed": "CUDA events around back-to-back launches of this call alone, after the timed region",
                    "peak_source": f"{peaks['source']} copy bandwidth"}
    per_call = {}
    for name in CALLS:
        sec = call_ms[name] * 1e-3
        per_call[name] = {"ms": call_ms[name], "GB/s": abytes[name] / sec / 1e9,
                          "frac_hbm": abytes[name] / sec / 1e9 / peaks["hbm_gbs"]}
    per_call["linear"]["TOPS"] = ops / (call_ms["linear"] * 1e-3) / 1e12
    per_call["linear"]["frac_int8_peak"] = per_call["linear"]["TOPS"] / int8_peak
    per_call["linear"]["ms_alone"] = call_ms_alone_linear

    # ---- the oracle on this machine's host cores, bounded sample ----------------------
    Ms, Ns = oracle_sample_shape(case)
    cpu_sec = oracle_step(case, Ms, Ns)
    cpu_value = layer_ops(Ms, Ns, K) / cpu_sec / 1e12
    sample = f"first {Ms} tokens x first {Ns} output channels, full K = {K}, whole path once ({cpu_sec:.1f} s)"

    line = {
        "metric": METRIC, "value": world * ops / (ms_per_step * 1e-3) / 1e12, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int4", "data": "synthetic",
        "config": {"workload": desc, "M": M, "N": N, "K": K, "calib_tokens": T, "alpha": case.alpha,
                   "step": "calibrate + fuse_weights + quant_act + linear",
                   "launch": "each step replays two CUDA graphs recorded from the C-ABI calls "
                             "([calibrate, fuse_weights, quant_act], [linear])",
                   "l2": f"inputs rotate through {n_sets} buffer sets ({n_sets * first.nbytes() / 2**20:.0f} MiB > 2 x L2)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "clocks": clocks,
        "e2e": {"value": world * ops / e2e_sec / 1e12, "unit": UNIT, "ms_per_step": e2e_sec * 1e3,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": sample},
        "per_call": per_call,
        "online_only": {"ms": call_ms["quant_act"] + call_ms["linear"],
                        "TOPS": ops / ((call_ms["quant_act"] + call_ms["linear"]) * 1e-3) / 1e12},
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="cfg1")
    args = ap.parse_args()
    maker, desc = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, maker(), desc)
        return
    run_gpu(args, maker(), desc)


if __name__ == "__main__":
    main()
