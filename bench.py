#!/usr/bin/env python
"""Benchmark of the SmoothRot W4A4 linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--per-config 0|1]
    python bench.py --workload cfg4 --shape gate_up --tokens 1 ...   # one point of the token-count sweep
    python bench.py --impl reference ...        # the CPU oracle on the host cores

One "step" is one pass of the whole path over one batch of seeded synthetic
input: calibrate (per-channel absmax -> scales), fuse_weights (scale, rotate,
quantize, pack W), quant_act (Hadamard + per-token INT4 quantize + pack X) and
linear (INT4 x INT4 GEMM + dequant to fp16).  The headline value is the layer's
2*M*N*K integer operations divided by the time of the whole step, on the
largest single-GPU workload (the fused gate/up projection, 8192 x 28672 x 4096).

The device-timed region keeps every input resident in HBM; between steps the
loop rotates through several distinct buffer sets whose total size exceeds
twice the L2 capacity, so no step finds its inputs in L2.  A step is launched
as two CUDA graphs recorded from the library calls, so that the Python cost of
a launch (longer than some of the kernels) does not sit in the device timeline;
a pair of events around the second graph times the GEMM kernel inside the
timed region.  After the K-step region the same region is repeated until half a
second of device time has been timed ("sustained": mean and minimum per step).
The end-to-end figure starts from pinned host buffers, makes the calls eagerly
and ends with the output back on the host, with the copies inside the timed
region.

The same run also measures an INT8 yardstick on the same GPU (a library int8
GEMM, 8192^3, burst and two seconds back to back) and, on one GPU, times every
call of the other workloads (`per_config`: the fused QKV projection, the
down-projection with the order-28 x Walsh-512 rotation, and a token-count sweep
over the linear shapes of one decoder block), each with its own clock record.

Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import re
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
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
METRIC = "w4a4_smoothrot_linear_tops"
UNIT = "TOPS"
SWEEP_TOKENS = (1, 16, 128, 512, 2048)

WORKLOADS = {
    "cfg0": (synth.config0, "configs[0]: tiny layer, X [64 x 128], W [256 x 128]"),
    "cfg1": (synth.config1, "configs[1]: LLaMA-3.1-8B-shaped fused QKV, X [2048 x 4096], W [6144 x 4096]"),
    "cfg2": (synth.config2, "configs[2]: down_proj with online Hadamard, X [2048 x 14336], W [4096 x 14336]"),
    "cfg3": (synth.config3, "configs[3]: fused gate/up projection (compute-bound GEMM), X [8192 x 4096], W [28672 x 4096]"),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TFLOPS, bf16_sustained=1400.0, source="fallback")


def profiled_traffic(M, N, K):
    """DRAM bytes (read + write) per launch of the GEMM kernel for this shape, from the tracked ncu
    summaries: a line `dram_bytes_per_launch M=.. N=.. K=..: <bytes>` in a file under profiles/.
    None when no summary covers the shape."""
    pat = re.compile(r"dram_bytes_per_launch\s+M=(\d+)\s+N=(\d+)\s+K=(\d+):\s*([0-9.eE+]+)")
    folder = os.path.join(ROOT, "profiles")
    if not os.path.isdir(folder):
        return None
    for name in sorted(os.listdir(folder)):
        if not name.endswith((".md", ".txt")):
            continue
        with open(os.path.join(folder, name)) as f:
            for m in pat.finditer(f.read()):
                if (int(m.group(1)), int(m.group(2)), int(m.group(3))) == (M, N, K):
                    return float(m.group(4))
    return None


def profiled_traffic_of(label):
    """Same, for a kernel that is not the GEMM: a line `dram_bytes_per_launch <label>: <bytes>`."""
    pat = re.compile(r"dram_bytes_per_launch\s+" + re.escape(label) + r":\s*([0-9.eE+]+)")
    folder = os.path.join(ROOT, "profiles")
    if not os.path.isdir(folder):
        return None
    for name in sorted(os.listdir(folder)):
        if name.endswith((".md", ".txt")):
            with open(os.path.join(folder, name)) as f:
                m = pat.search(f.read())
                if m:
                    return float(m.group(1))
    return None


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
    """Samples nvidia-smi clocks and throttle reasons while a timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, enabled: bool = True):
        self.index = index
        self.enabled = enabled
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        if not self.enabled:
            return self
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return self
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def mark(self):
        return time.perf_counter()

    def stop(self, since=None, until=None):
        """Summary of the samples taken between the two marks (all samples if none given)."""
        if not self.enabled:
            return None
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self.summary(since, until)

    def summary(self, since=None, until=None):
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, line in list(self.lines):
            if since is not None and stamp < since:
                continue
            if until is not None and stamp > until + 0.06:
                continue
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
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_min_mhz": float(min(sm)), "sm_max_mhz": float(max(smax)),
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

    def __init__(self, torch, sr, case, dev, M=None):
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        M = case.M if M is None else M
        N, K = case.N, case.K
        self.M = M
        self.X, self.Xc, self.W, self.d = t(case.X[:M]), t(case.X_calib), t(case.W), t(case.d)
        f32 = lambda n: torch.empty(n, dtype=torch.float32, device=dev)
        self.amax, self.s, self.pre_w, self.pre_x = f32(K), f32(K), f32(K), f32(K)
        self.wq = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
        self.xq = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
        self.xq2 = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)   # outputs of the call without a diagonal
        self.dw, self.dx, self.dx2 = f32(N), f32(M), f32(M)
        self.Y = torch.empty((M, N), dtype=torch.float16, device=dev)
        need = sr.workspace_bytes(M, N, K)
        self.ws = torch.empty(need, dtype=torch.uint8, device=dev) if need else None

    def nbytes(self):
        tensors = (self.X, self.Xc, self.W, self.wq, self.xq, self.Y)
        return sum(x.numel() * x.element_size() for x in tensors)

    def online_nbytes(self):
        tensors = (self.X, self.wq, self.xq, self.Y)
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
        # not a step of the path: the exact online Hadamard of the paper's deployment (Lambda^-1 absorbed
        # by the producing layer, no sign diagonal), timed beside quant_act for comparison
        "quant_act_exact": lambda: sr.quant_act(ds.X, None, case.clip_a, ds.xq2, ds.dx2),
    }


def gpu_step(sr, case, ds):
    """The whole path on one buffer set, call by call (eager launches)."""
    calls = step_calls(sr, case, ds)
    for name in CALLS:
        calls[name]()


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


def time_replays(torch, graphs, min_seconds=0.2, reps=20, max_regions=4000):
    """Replays the graphs round robin, `reps` replays per event-bracketed region, region after
    region until `min_seconds` of device time have been timed.  Returns (mean, minimum) seconds
    per replay over the regions and the number of regions."""
    n = len(graphs)
    for i in range(max(3, n)):
        graphs[i % n].replay()
    torch.cuda.synchronize()
    per, total, k = [], 0.0, 0
    while total < min_seconds and len(per) < max_regions:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            graphs[k % n].replay()
            k += 1
        e1.record()
        torch.cuda.synchronize()
        sec = e0.elapsed_time(e1) * 1e-3
        per.append(sec / reps)
        total += sec
    return float(np.mean(per)), float(np.min(per)), len(per)


def int8_yardstick(torch, dev, seconds=2.0):
    """An int8 tensor-core GEMM from the vendor library on this GPU's own memory (8192^3, int32
    accumulation): best of ten single calls ("burst") and the mean rate of calls back to back for
    `seconds` ("sustained").  A yardstick for the roofline's denominator only; no part of the path."""
    n = 8192
    try:
        a = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=dev)
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch._int_mm(a, b); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) * 1e-3)
        ops = 2.0 * n ** 3
        calls, total = 0, 0.0
        while total < seconds:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(20):
                torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1) * 1e-3
            calls += 20
        del a, b
        return {"burst_tops": ops / best / 1e12, "sustained_tops": ops * calls / total / 1e12,
                "how": f"library int8 GEMM {n}^3, best of 10 / {calls} calls back to back ({total:.1f} s)"}
    except Exception as exc:   # the yardstick is optional: report why it is missing
        return {"burst_tops": None, "sustained_tops": None, "how": f"unavailable: {type(exc).__name__}: {exc}"}


def peaks_record(peaks, yard):
    rec = {
        "hbm_gbs": peaks["hbm_gbs"], "hbm_source": f"{peaks['source']} copy bandwidth", "hbm_nominal_gbs": NOMINAL_HBM_GBS,
        "int8_from_bf16_burst": peaks["bf16"] * 2.0, "int8_from_bf16_sustained": peaks["bf16_sustained"] * 2.0,
        "int8_nominal": NOMINAL_INT8_TOPS,
        "int8_measured_in_run_burst": yard["burst_tops"], "int8_measured_in_run_sustained": yard["sustained_tops"],
        "int8_measured_how": yard["how"],
    }
    return rec


def linear_fracs(tops, rec):
    out = {"of_bf16_burst_x2": tops / rec["int8_from_bf16_burst"],
           "of_bf16_sustained_x2": tops / rec["int8_from_bf16_sustained"],
           "of_nominal_4500": tops / rec["int8_nominal"]}
    if rec["int8_measured_in_run_burst"]:
        out["of_int8_measured_burst"] = tops / rec["int8_measured_in_run_burst"]
        out["of_int8_measured_sustained"] = tops / rec["int8_measured_in_run_sustained"]
    return out


def measure_layer(torch, sr, case, dev, rec, local, min_seconds, sampler_on=True):
    """Every call of the path on one workload, each alone (graph replays, buffer sets rotated out
    of L2), plus the whole step; with a clock record of its own."""
    M, N, K, T = case.M, case.N, case.K, case.X_calib.shape[0]
    first = DeviceSet(torch, sr, case, dev)
    n_sets = max(2, int(np.ceil(2.2 * L2_BYTES / first.nbytes())))
    sets = [first] + [DeviceSet(torch, sr, case, dev) for _ in range(1, n_sets)]
    for ds in sets:
        gpu_step(sr, case, ds)
    torch.cuda.synchronize()
    graphs = {name: [] for name in CALLS}
    whole = []
    for ds in sets:
        calls = step_calls(sr, case, ds)
        for name in CALLS:
            graphs[name].append(capture(torch, [calls[name]]))
        whole.append(capture(torch, [calls[name] for name in CALLS]))
    sampler = ClockSampler(local, sampler_on).start()
    abytes = algorithmic_bytes(M, N, K, T)
    out = {"M": M, "N": N, "K": K, "buffer_sets": n_sets, "linear_kernel": sr.linear_plan_name(M, N, K)}
    for name in CALLS:
        mean, best, regions = time_replays(torch, graphs[name], min_seconds)
        entry = {"us": mean * 1e6, "us_min": best * 1e6, "regions": regions,
                 "GB/s": abytes[name] / mean / 1e9, "frac_hbm": abytes[name] / mean / 1e9 / rec["hbm_gbs"]}
        if name == "linear":
            tops = layer_ops(M, N, K) / mean / 1e12
            entry["TOPS"] = tops
            entry["frac"] = linear_fracs(tops, rec)
        out[name] = entry
    exact = [capture(torch, [step_calls(sr, case, ds)["quant_act_exact"]]) for ds in sets]
    mean, best, regions = time_replays(torch, exact, min_seconds)
    out["quant_act_exact"] = {"us": mean * 1e6, "us_min": best * 1e6, "GB/s": abytes["quant_act"] / mean / 1e9,
                              "frac_hbm": abytes["quant_act"] / mean / 1e9 / rec["hbm_gbs"],
                              "note": "smoothrot_quant_act without a diagonal (exact online Hadamard); not part of the step"}
    mean, best, regions = time_replays(torch, whole, min_seconds)
    out["step"] = {"us": mean * 1e6, "us_min": best * 1e6, "TOPS": layer_ops(M, N, K) / mean / 1e12}
    out["clocks"] = sampler.stop()
    assert sr.device_status() == 0, "a device-side wait timed out"
    del graphs, whole, sets, first
    torch.cuda.empty_cache()
    return out


def measure_sweep(torch, sr, dev, rec, local, min_seconds, sampler_on=True):
    """The online calls (quant_act, linear) of every linear shape of one decoder block at several
    token counts, from decode to prefill; weights quantized once per shape; inputs, codes, weights
    and outputs rotated out of L2."""
    rows = []
    for name, N, K in synth.BLOCK_SHAPES:
        case = synth.config4(name, max(SWEEP_TOKENS))     # rows 0..M-1 of one draw serve every M
        full = DeviceSet(torch, sr, case, dev)
        gpu_step(sr, case, full)
        torch.cuda.synchronize()
        sampler = ClockSampler(local, sampler_on).start()
        shape_rows = []
        for M in SWEEP_TOKENS:
            per_set = N * K // 2 + M * K * 2 + M * K // 2 + M * N * 2
            n_sets = int(min(24, max(2, np.ceil(2.2 * L2_BYTES / per_set))))
            sets = []
            for _ in range(n_sets):
                X = full.X[:M].clone()
                wq, dw = full.wq.clone(), full.dw.clone()
                xq = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
                dx = torch.empty(M, dtype=torch.float32, device=dev)
                Y = torch.empty((M, N), dtype=torch.float16, device=dev)
                need = sr.workspace_bytes(M, N, K)
                ws = torch.empty(need, dtype=torch.uint8, device=dev) if need else None
                sr.quant_act(X, full.pre_x, case.clip_a, xq, dx)
                sr.linear(xq, dx, wq, dw, Y, ws)
                sets.append((X, xq, dx, wq, dw, Y, ws))
            torch.cuda.synchronize()
            gq = [capture(torch, [lambda s=s: sr.quant_act(s[0], full.pre_x, case.clip_a, s[1], s[2])]) for s in sets]
            gl = [capture(torch, [lambda s=s: sr.linear(s[1], s[2], s[3], s[4], s[5], s[6])]) for s in sets]
            ge = [capture(torch, [lambda s=s: sr.quant_act(s[0], None, case.clip_a, s[1], s[2])]) for s in sets]
            te, te_min, _ = time_replays(torch, ge, min_seconds)
            tq, tq_min, _ = time_replays(torch, gq, min_seconds)
            tl, tl_min, _ = time_replays(torch, gl, min_seconds)
            ops = layer_ops(M, N, K)
            row = {"shape": name, "N": N, "K": K, "M": M, "buffer_sets": n_sets,
                   "linear_kernel": sr.linear_plan_name(M, N, K),
                   "quant_act_us": tq * 1e6, "quant_act_us_min": tq_min * 1e6,
                   "quant_act_GBs": (2.5 * M * K + 4 * M + 4 * K) / tq / 1e9,
                   "quant_act_exact_us": te * 1e6, "quant_act_exact_GBs": (2.5 * M * K + 4 * M) / te / 1e9,
                   "linear_us": tl * 1e6, "linear_us_min": tl_min * 1e6, "linear_TOPS": ops / tl / 1e12,
                   "linear_frac_bf16_burst_x2": ops / tl / 1e12 / rec["int8_from_bf16_burst"],
                   "weight_stream_GBs": 0.5 * N * K / tl / 1e9,
                   "weight_stream_frac_hbm": 0.5 * N * K / tl / 1e9 / rec["hbm_gbs"],
                   "algorithmic": {"ops": ops, "linear_bytes": 0.5 * M * K + 0.5 * N * K + 2.0 * M * N + 4.0 * (M + N),
                                   "quant_act_bytes": 2.5 * M * K + 4 * M + 4 * K}}
            shape_rows.append(row)
            del sets, gq, gl, ge
            torch.cuda.empty_cache()
        clocks = sampler.stop()
        for row in shape_rows:
            row["clocks"] = clocks
        rows.extend(shape_rows)
        assert sr.device_status() == 0, "a device-side wait timed out"
        del full
        torch.cuda.empty_cache()
    return rows


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

    def timed_region(steps, with_events):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)] if with_events else None
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for i in range(steps):
            front[i % n_sets].replay()
            if with_events:
                ev[i][0].record()
            back[i % n_sets].replay()
            if with_events:
                ev[i][1].record()
        stop.record()
        barrier()
        total_ms = max_over_ranks(torch, dist, start.elapsed_time(stop), dev)
        lin = float(np.mean([a.elapsed_time(b) for a, b in ev])) if with_events else None
        return total_ms, lin

    # ---- device-timed region: exactly K steps ---------------------------------------
    sampler = ClockSampler(local, rank == 0).start()
    t_a = sampler.mark()
    total_ms, linear_live_ms = timed_region(args.steps, True)
    t_b = sampler.mark()
    launches = launches_per_step * args.steps
    ms_per_step = total_ms / args.steps
    assert sr.device_status() == 0, "a device-side wait timed out"

    # ---- the same region again and again until half a second of device time is covered ----
    regions, covered = [ms_per_step], total_ms
    while covered < args.min_region_s * 1e3 and len(regions) < 2000:
        t_ms, _ = timed_region(args.steps, False)
        regions.append(t_ms / args.steps)
        covered += t_ms
    t_c = sampler.mark()
    # one record over the K-step region and its repeats (the same work; the first region alone can
    # be shorter than the sampling interval), with the number of samples that fell into the first
    clocks = sampler.stop(t_a, t_c) if rank == 0 else None
    if clocks is not None:
        clocks["samples_in_first_region"] = (sampler.summary(t_a, t_b) or {}).get("samples", 0)
        clocks["covers"] = "the K-step region and its repeats (sustained)"

    # ---- each call alone (outside the timed region): one graph per call and buffer set ----
    call_ms, call_ms_min = {}, {}
    sampler2 = ClockSampler(local, rank == 0).start()
    for name in CALLS:
        mean, best, _ = time_replays(torch, single[name], 0.25 if name == "linear" else 0.1)
        call_ms[name], call_ms_min[name] = mean * 1e3, best * 1e3
    for ds in sets:
        step_calls(sr, case, ds)["quant_act_exact"]()
    torch.cuda.synchronize()
    exact_graphs = [capture(torch, [step_calls(sr, case, ds)["quant_act_exact"]]) for ds in sets]
    exact_mean, exact_min, _ = time_replays(torch, exact_graphs, 0.1)
    clocks_calls = sampler2.stop() if rank == 0 else None
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
    del host_in, host_Y

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- the denominators: measured copy bandwidth, bf16-derived and in-run int8 rates ----
    peaks = measured_peaks()
    yard = int8_yardstick(torch, dev)
    rec = peaks_record(peaks, yard)

    ops = layer_ops(M, N, K)
    int8_peak = rec["int8_from_bf16_burst"]
    abytes = algorithmic_bytes(M, N, K, T)
    dominant = max(call_ms, key=call_ms.get)
    if dominant == "linear":
        achieved = ops / (call_ms["linear"] * 1e-3) / 1e12
        traffic = profiled_traffic(M, N, K)
        roofline = {"kernel": f"{sr.linear_plan_name(M, N, K)} (smoothrot_linear)", "bound": "tensor",
                    "achieved": achieved, "peak": int8_peak, "unit": "TOP/s", "frac": achieved / int8_peak,
                    "traffic": traffic,
                    "traffic_note": ("dram read + write bytes of one launch from the ncu summary under profiles/; "
                                     "part of Y may still sit in L2 when the kernel ends") if traffic else
                                    "no ncu summary under profiles/ covers this shape",
                    "algorithmic_ops": ops, "algorithmic_bytes": abytes["linear"],
                    "timed": "CUDA events around the kernel's launch inside the timed region, mean over the steps",
                    "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16']} TFLOP/s x 2 (nominal int8:bf16 ratio)",
                    "fracs": linear_fracs(achieved, rec)}
    else:
        achieved = abytes[dominant] / (call_ms[dominant] * 1e-3) / 1e9
        roofline = {"kernel": dominant, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                    "timed": "CUDA events around back-to-back launches of this call alone, after the timed region",
                    "peak_source": f"{peaks['source']} copy bandwidth"}
    per_call = {}
    for name in CALLS:
        sec = call_ms[name] * 1e-3
        per_call[name] = {"ms": call_ms[name], "ms_min_alone": call_ms_min[name], "GB/s": abytes[name] / sec / 1e9,
                          "frac_hbm": abytes[name] / sec / 1e9 / peaks["hbm_gbs"],
                          "frac_hbm_nominal_8000": abytes[name] / sec / 1e9 / NOMINAL_HBM_GBS,
                          "algorithmic_bytes": abytes[name]}
    per_call["linear"]["TOPS"] = ops / (call_ms["linear"] * 1e-3) / 1e12
    per_call["linear"]["frac_int8_peak"] = per_call["linear"]["TOPS"] / int8_peak
    per_call["linear"]["ms_alone"] = call_ms_alone_linear
    per_call["quant_act_exact"] = {
        "ms": exact_mean * 1e3, "ms_min_alone": exact_min * 1e3, "GB/s": abytes["quant_act"] / exact_mean / 1e9,
        "frac_hbm": abytes["quant_act"] / exact_mean / 1e9 / peaks["hbm_gbs"],
        "frac_hbm_nominal_8000": abytes["quant_act"] / exact_mean / 1e9 / NOMINAL_HBM_GBS,
        "note": "smoothrot_quant_act without a diagonal (the exact online Hadamard of the paper's deployment, "
                "Lambda^-1 absorbed by the producing layer); timed alone, not part of the step"}
    per_call["clocks"] = clocks_calls

    # the memory-bound kernel of the online path, against the copy bandwidth
    def hbm_roofline(kernel, seconds, label):
        got = abytes["quant_act"] / seconds / 1e9
        return {"kernel": kernel, "bound": "hbm", "achieved": got, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": got / peaks["hbm_gbs"], "traffic": profiled_traffic_of(label),
                "algorithmic_bytes": abytes["quant_act"],
                "timed": "CUDA events around back-to-back launches of this call alone, inputs rotated out of L2",
                "peak_source": f"{peaks['source']} copy bandwidth"}
    roofline_quant = {
        "diagonal": hbm_roofline("smoothrot_quant_act, diagonal d/s (register kernel)", call_ms["quant_act"] * 1e-3,
                                 f"quant_act rows={M} K={K} diagonal=1"),
        "no_diagonal": hbm_roofline("smoothrot_quant_act, no diagonal", exact_mean,
                                    f"quant_act rows={M} K={K} diagonal=0")}

    # ---- the other workloads, one GPU only (each with its own clock record) ----
    per_config = None
    if args.per_config and world == 1:
        del front, back, single, sets, first
        torch.cuda.empty_cache()
        per_config = {}
        for key in ("cfg1", "cfg2"):
            if key == args.workload:
                continue
            maker, d2 = WORKLOADS[key]
            per_config[key] = measure_layer(torch, sr, maker(), dev, rec, local, args.min_config_s)
            per_config[key]["workload"] = d2
        per_config["cfg4_sweep"] = measure_sweep(torch, sr, dev, rec, local, args.min_config_s)

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
                   "l2": f"inputs rotate through {n_sets} buffer sets ({n_sets * first_bytes(M, N, K, T) / 2**20:.0f} MiB > 2 x L2)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "clocks": clocks,
        "sustained": {"ms_per_step_mean": float(np.mean(regions)), "ms_per_step_min": float(np.min(regions)),
                      "regions": len(regions), "device_seconds": covered * 1e-3,
                      "TOPS_mean": world * ops / (float(np.mean(regions)) * 1e-3) / 1e12},
        "e2e": {"value": world * ops / e2e_sec / 1e12, "unit": UNIT, "ms_per_step": e2e_sec * 1e3,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "roofline_quant_act": roofline_quant,
        "peaks": rec,
        "cpu_baseline": {"value": cpu_value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": sample},
        "per_call": per_call,
        "online_only": {"ms": call_ms["quant_act"] + call_ms["linear"],
                        "TOPS": ops / ((call_ms["quant_act"] + call_ms["linear"]) * 1e-3) / 1e12},
    }
    if per_config is not None:
        line["per_config"] = per_config
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def first_bytes(M, N, K, T):
    """Bytes of one buffer set (inputs, codes, output)."""
    return 2 * M * K + 2 * T * K + 2 * N * K + N * K // 2 + M * K // 2 + 2 * M * N


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS) + ["cfg4"], default="cfg3")
    ap.add_argument("--shape", choices=[n for n, _, _ in synth.BLOCK_SHAPES], default="gate_up",
                    help="with --workload cfg4: the linear shape of the decoder block")
    ap.add_argument("--tokens", type=int, default=1, help="with --workload cfg4: the token count M")
    ap.add_argument("--per-config", type=int, default=1, help="0: skip the records of the other workloads")
    ap.add_argument("--min-region-s", type=float, default=0.5,
                    help="device seconds the repeated K-step regions must cover")
    ap.add_argument("--min-config-s", type=float, default=0.06,
                    help="device seconds per timed call in the per-config records")
    args = ap.parse_args()
    if args.workload == "cfg4":
        maker = lambda: synth.config4(args.shape, args.tokens)
        desc = f"configs[4]: one point of the token-count sweep, shape {args.shape}, M = {args.tokens}"
    else:
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
