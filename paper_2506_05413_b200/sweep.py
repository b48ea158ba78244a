"""Token-count sweep over the linear shapes of one LLaMA-3.1-8B-shaped decoder block.

    python -m paper_2506_05413_b200.sweep [--reps 30] [--json] [--shapes ...] [--tokens ...]
    python -m paper_2506_05413_b200.sweep --kv        # the KV-cache codec instead

For every shape (q/o 4096->4096, k/v 4096->1024, gate/up 4096->14336, down 14336->4096) and
every M in {1, 4, 16, 128, 512, 2048, 8192} it times the two online calls of the layer,
smoothrot_quant_act and smoothrot_linear, on seeded synthetic activations (random-init
weights, quantized once by smoothrot_fuse_weights), and prints time, TOP/s and GB/s; for the q/o
shape also smoothrot_quant_act_heads (32 heads of 128), the transform the o-projection's input takes,
and for K = 4096 smoothrot_linear_decode, which does both calls in one kernel (M <= 4 with the
rotation: "fused"; M <= 8 without: "fusedP"; M <= 4 with the head mixing, q/o shape: "fusedH").

Timing: each call is recorded into a CUDA graph per buffer set and replayed back to back
between two CUDA events; the buffer sets rotate so that their total size exceeds twice the
L2 capacity (weights included), which is what a decode step of a whole model sees.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import synth

L2_BYTES = 126 * 1024 * 1024
HEADS = 32          # 32 heads of 128: the attention output of the 8B-class models


def _time_graphs(torch, graphs, reps):
    n = len(graphs)
    for i in range(max(3, n)):
        graphs[i % n].replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        graphs[i % n].replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / reps      # seconds


def run(reps: int = 30, shapes=None, tokens=None):
    import torch
    from . import binding as sr

    sr.load()
    dev = "cuda:0"
    rows = []
    for name, N, K in synth.BLOCK_SHAPES:
        if shapes and name not in shapes:
            continue
        base = synth.config4(name, 8)                      # weights and diagonal do not depend on M
        W = torch.from_numpy(base.W).to(dev)
        d = torch.from_numpy(base.d).to(dev)
        Xc = torch.from_numpy(base.X_calib).to(dev)
        amax = torch.zeros(K, dtype=torch.float32, device=dev)
        s, pre_w, pre_x = (torch.empty(K, dtype=torch.float32, device=dev) for _ in range(3))
        sr.calibrate(Xc, amax, W=W, alpha=base.alpha, s_out=s, d=d, pre_w_out=pre_w, pre_x_out=pre_x)
        for M in (tokens or synth.SWEEP_M):
            case = synth.config4(name, M)
            per_set = N * K // 2 + M * K * 2 + M * K // 2 + M * N * 2
            n_sets = int(min(24, max(2, np.ceil(2.2 * L2_BYTES / per_set))))
            sets = []
            for _ in range(n_sets):
                wq = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
                dw = torch.empty(N, dtype=torch.float32, device=dev)
                sr.fuse_weights(W, pre_w, case.clip_w, wq, dw)
                X = torch.from_numpy(case.X).to(dev)
                xq = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
                dx = torch.empty(M, dtype=torch.float32, device=dev)
                Y = torch.empty((M, N), dtype=torch.float16, device=dev)
                need = sr.workspace_bytes(M, N, K)
                ws = torch.empty(need, dtype=torch.uint8, device=dev) if need else None
                sr.quant_act(X, pre_x, case.clip_a, xq, dx)
                sr.linear(xq, dx, wq, dw, Y, ws)
                sets.append((X, xq, dx, wq, dw, Y, ws))
            torch.cuda.synchronize()
            gq, gl, gh, gf, gp, gfp, gfh = [], [], [], [], [], [], []
            for X, xq, dx, wq, dw, Y, ws in sets:
                sr.quant_act_plain(X, pre_x, case.clip_a, xq, dx)       # the quantizer without a rotation
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    sr.quant_act_plain(X, pre_x, case.clip_a, xq, dx)
                gp.append(g)
                if M <= 8 and K == 4096:    # the same without a rotation
                    sr.linear_decode(X, pre_x, case.clip_a, wq, dw, Y, rotation=False)
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        sr.linear_decode(X, pre_x, case.clip_a, wq, dw, Y, rotation=False)
                    gfp.append(g)
                if M <= 4 and name == "q_o":    # the o-projection's layer: head mixing + linear in one kernel
                    sr.linear_decode_heads(X, HEADS, None, case.clip_a, wq, dw, Y)
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        sr.linear_decode_heads(X, HEADS, None, case.clip_a, wq, dw, Y)
                    gfh.append(g)
                if M <= 4 and K == 4096:    # both calls of the layer in one kernel
                    sr.linear_decode(X, pre_x, case.clip_a, wq, dw, Y)
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        sr.linear_decode(X, pre_x, case.clip_a, wq, dw, Y)
                    gf.append(g)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    sr.quant_act(X, pre_x, case.clip_a, xq, dx)
                gq.append(g)
                if name == "q_o":      # the o-projection's input also has the head-mixing variant
                    sr.quant_act_heads(X, HEADS, None, case.clip_a, xq, dx)
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        sr.quant_act_heads(X, HEADS, None, case.clip_a, xq, dx)
                    gh.append(g)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    sr.linear(xq, dx, wq, dw, Y, ws)
                gl.append(g)
            tl = _time_graphs(torch, gl, reps)
            th = _time_graphs(torch, gh, reps) if gh else None
            tf = _time_graphs(torch, gf, reps) if gf else None
            tp = _time_graphs(torch, gp, reps)
            tfp = _time_graphs(torch, gfp, reps) if gfp else None
            tfh = _time_graphs(torch, gfh, reps) if gfh else None
            tq = _time_graphs(torch, gq, reps)
            assert sr.device_status() == 0
            ops = 2.0 * M * N * K
            rows.append({
                "shape": name, "N": N, "K": K, "M": M,
                "quant_act_us": tq * 1e6, "quant_act_GBs": (2.5 * M * K + 4 * M + 4 * K) / tq / 1e9,
                "linear_us": tl * 1e6, "linear_TOPS": ops / tl / 1e12,
                "linear_GBs": (0.5 * M * K + 0.5 * N * K + 2.0 * M * N + 4 * (M + N)) / tl / 1e9,
                "weight_stream_GBs": 0.5 * N * K / tl / 1e9,
                "buffer_sets": n_sets,
            })
            rows[-1]["quant_act_plain_us"] = tp * 1e6
            rows[-1]["quant_act_plain_GBs"] = (2.5 * M * K + 4 * M + 4 * K) / tp / 1e9
            if tf is not None:
                rows[-1]["fused_layer_us"] = tf * 1e6
            if tfp is not None:
                rows[-1]["fused_plain_layer_us"] = tfp * 1e6
            if tfh is not None:
                rows[-1]["fused_heads_layer_us"] = tfh * 1e6
            if th is not None:
                rows[-1]["quant_act_heads_us"] = th * 1e6
                rows[-1]["quant_act_heads_GBs"] = (2.5 * M * K + 4 * M) / th / 1e9
            del sets, gq, gl
            torch.cuda.empty_cache()
    return rows


def run_kv(reps: int = 30, rows: int = 65536, width: int = 1024):
    """Times the KV-cache codec (smoothrot_kv_quant / smoothrot_kv_dequant) on `rows` cache rows of
    `width` values (8 KV heads of 128), two buffer sets of seeded N(0,1) values, each larger than L2."""
    import torch
    from . import binding as sr

    sr.load()
    dev = "cuda:0"
    rng = np.random.default_rng(7)
    host = torch.from_numpy(rng.standard_normal((rows, width), dtype=np.float32).astype(np.float16))
    sets = []
    for _ in range(2):
        X = host.to(dev)
        q = torch.empty((rows, width // 2), dtype=torch.uint8, device=dev)
        step = torch.empty((rows, width // 128), dtype=torch.float32, device=dev)
        zero = torch.empty_like(step)
        Y = torch.empty_like(X)
        sr.kv_quant(X, 0.95, q, step, zero)
        sr.kv_dequant(q, step, zero, Y)
        sets.append((X, q, step, zero, Y))
    torch.cuda.synchronize()
    gq, gd = [], []
    for X, q, step, zero, Y in sets:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            sr.kv_quant(X, 0.95, q, step, zero)
        gq.append(g)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            sr.kv_dequant(q, step, zero, Y)
        gd.append(g)
    tq = _time_graphs(torch, gq, reps)
    td = _time_graphs(torch, gd, reps)
    n = rows * width
    bytes_per_call = n * (2 + 0.5 + 8 / 128)
    return {"rows": rows, "width": width, "kv_quant_us": tq * 1e6, "kv_quant_GBs": bytes_per_call / tq / 1e9,
            "kv_dequant_us": td * 1e6, "kv_dequant_GBs": bytes_per_call / td / 1e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--json", action="store_true")
    ap.add_argument("--shapes", nargs="*")
    ap.add_argument("--tokens", nargs="*", type=int)
    ap.add_argument("--kv", action="store_true", help="time the KV-cache codec instead of the linear shapes")
    args = ap.parse_args()
    if args.kv:
        print(json.dumps(run_kv(args.reps)))
        return
    rows = run(args.reps, args.shapes, args.tokens)
    if args.json:
        for r in rows:
            print(json.dumps(r))
        return
    print(f"{'shape':8s} {'M':>5s} {'quant us':>9s} {'GB/s':>7s} {'plain us':>9s} {'GB/s':>7s} {'linear us':>10s} {'TOP/s':>8s} {'W GB/s':>8s}"
          f" {'heads us':>9s} {'GB/s':>7s} {'fused us':>9s} {'fusedP us':>9s} {'fusedH us':>9s}")
    for r in rows:
        heads = (f" {r['quant_act_heads_us']:9.1f} {r['quant_act_heads_GBs']:7.0f}"
                 if "quant_act_heads_us" in r else " " * 18)
        heads += f" {r['fused_layer_us']:9.1f}" if "fused_layer_us" in r else " " * 10
        heads += f" {r['fused_plain_layer_us']:9.1f}" if "fused_plain_layer_us" in r else " " * 10
        if "fused_heads_layer_us" in r:
            heads += f" {r['fused_heads_layer_us']:9.1f}"
        print(f"{r['shape']:8s} {r['M']:5d} {r['quant_act_us']:9.1f} {r['quant_act_GBs']:7.0f} "
              f"{r['quant_act_plain_us']:9.1f} {r['quant_act_plain_GBs']:7.0f} "
              f"{r['linear_us']:10.1f} {r['linear_TOPS']:8.1f} {r['weight_stream_GBs']:8.0f}{heads}")


if __name__ == "__main__":
    main()
