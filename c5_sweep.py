"""Skewed-routing token sweep (workload C5): DeepSeek-V3-shaped layer, Zipf(1.2) expert popularity,
T in {1, 16, 128, 1024, 8192, 32768}.  For every T: layer time and tokens/s, per-stage device times, expert
load imbalance, and the fraction of the layer's roofline floor that was reached.

    python c5_sweep.py [--tokens 1 16 128 ...] [--iters-min-ms 300] [--fp8]
    python c5_sweep.py --route-only [--tokens ...]     # stage a1 by itself (no weights are allocated)

One JSON object per T on stdout.  The floor of a step is the sum over its stages of
max(flops / tensor peak, algorithmic bytes / HBM peak); for the grouped GEMMs it is summed per expert
(a cold expert is bound by streaming its weights, a hot one by the tensor cores).  Peaks come from
MEASURED_PEAKS.json at the repository root when present (HBM copy GB/s, sustained bf16 TFLOP/s).
"""
from __future__ import annotations

import argparse
import json
import os

import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return d["hbm_gbs"], d.get("bf16_tflops_sustained", d["bf16_tflops"]), "measured"
    return 6650.0, 1400.0, "fallback"


def layer_floor_us(shape, counts, hbm_gbs, tflops, fp8=False):
    """Roofline floor of one step in microseconds, and its tensor-only / bytes-only parts.  FP8: one byte per
    weight and per GEMM input element, and twice the bf16 tensor peak (the nominal fp8 : bf16 ratio)."""
    H, I, k, T = shape.H, shape.I, shape.k, shape.T
    bw, peak = hbm_gbs * 1e9, tflops * 1e12 * (2.0 if fp8 else 1.0)
    eb = 1.0 if fp8 else 2.0  # bytes per operand element
    gemm = fl_only = by_only = 0.0
    groups = [(int(c), I) for c in counts.tolist() if c > 0]
    if shape.shared_I:
        groups.append((T, shape.shared_I))
    for rows, inter in groups:
        flops = 6.0 * rows * H * inter
        # weights, rows in, act written (bf16) and read (FP8: re-quantised: bf16 read + codes written + codes read), out
        act = (2.0 + 2.0 + 1.0 + 1.0) * rows * inter if fp8 else 4.0 * rows * inter
        bytes_ = 3.0 * eb * H * inter + eb * rows * H + act + 2.0 * rows * H
        gemm += max(flops / peak, bytes_ / bw)
        fl_only += flops / peak
        by_only += bytes_ / bw
    N = T * k
    rows_in = (2.0 * T * H + 1.0 * T * H) + (1.0 * T * H + 1.0 * N * H + 8.0 * N) if fp8 else 2.0 * T * H + 2.0 * N * H + 4.0 * N
    rows_bytes = rows_in + (2.0 * N * H + 2.0 * bool(shape.shared_I) * T * H + 8.0 * N + 2.0 * T * H)
    route_bytes = 4.0 * T * shape.E + 8.0 * N + 12.0 * N
    other = (rows_bytes + route_bytes) / bw
    return 1e6 * (gemm + other), 1e6 * fl_only, 1e6 * by_only


def run_one(shape, weights, min_ms, dev="cuda", fp8=False):
    phase = B.MOE_PHASE_DECODE if shape.T <= 256 else B.MOE_PHASE_PREFILL
    stream = torch.cuda.Stream()
    fmt = B.MOE_WEIGHTS_FP8_E4M3 if fp8 else B.MOE_WEIGHTS_BF16
    ctx = B.MoeContext(B.make_config(shape.H, shape.E, shape.k, shape.I, shape.shared_I, shape.T, phase,
                                     weight_format=fmt), stream=stream)
    acts = [wl.make_activations(shape, 600 + i, dev) for i in range(3)]
    bufs = B.alloc_step_buffers(shape.T, shape.k, shape.E, dev)
    out = torch.empty(shape.T, shape.H, dtype=torch.bfloat16, device=dev)

    def step(i):
        a = acts[i % 3]
        if fp8:
            ctx.layer_fp8(a["x"], a["logits"], a["bias"], weights, out=out, bufs=bufs)
        else:
            ctx.layer(a["x"], a["logits"], a["bias"], weights["w_gate_up"], weights["w_down"], weights["ws_gate_up"],
                      weights["ws_down"], out=out, bufs=bufs)

    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for i in range(5):
            step(i)
    torch.cuda.synchronize()
    n, total_ms = 4, 0.0
    while True:
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(n):
                step(i)
            e1.record(stream)
        torch.cuda.synchronize()
        total_ms = e0.elapsed_time(e1)
        if total_ms >= min_ms or n >= 4096:
            break
        n *= 2
    step_us = 1e3 * total_ms / n
    ctx.moe_ctx_set_profiling(True)
    with torch.cuda.stream(stream):
        for i in range(min(n, 32)):
            step(i)
    prof = ctx.moe_ctx_read_profile()
    ctx.moe_ctx_set_profiling(False)
    assert ctx.moe_ctx_status() == B.MOE_OK
    counts = bufs["counts"].cpu()
    ctx.close()
    return step_us, n, {k_: round(1e3 * ms / c, 1) for k_, (ms, c) in prof.items() if c}, counts


def route_only(tokens, E, k, zipf, hbm, src, launches=200):
    """Stage a1 by itself on the sweep's logits: microseconds per launch (back to back on one stream, so the figure
    includes the launch rate of tiny problems) and the achieved fraction of the HBM copy rate."""
    dev = "cuda"
    for T in tokens:
        shape = wl.LayerShape("route", T=T, H=64, E=E, k=k, I=64, zipf_s=zipf, select_bias=zipf == 0)
        acts = [wl.make_activations(shape, 600 + i, dev) for i in range(3)]
        stream = torch.cuda.Stream()
        ctx = B.MoeContext(B.make_config(64, E, k, 64, 0, T, B.MOE_PHASE_PREFILL), stream=stream)
        idx = torch.empty(T, k, dtype=torch.int32, device=dev)
        w = torch.empty(T, k, dtype=torch.float32, device=dev)

        def run(n):
            for i in range(n):
                a = acts[i % 3]
                ctx.moe_route(a["logits"], a["bias"], idx, w)
                ctx.moe_ctx_abandon_step()

        with torch.cuda.stream(stream):
            run(5)
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run(launches)
            e1.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / launches
        by = 4.0 * T * E + 4.0 * E + 8.0 * T * k
        assert ctx.moe_ctx_status() == B.MOE_OK
        ctx.close()
        print(json.dumps({"workload": f"route only, E={E} top-{k} T={T}", "us_per_launch": round(us, 2),
                          "algorithmic_bytes": by, "GBps": round(by / us / 1e3, 1),
                          "frac_hbm": round(by / us / 1e3 / hbm, 3), "peak_source": src}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, nargs="*", default=list(wl.C5_TOKENS))
    ap.add_argument("--iters-min-ms", type=float, default=300.0, help="time each T for at least this long")
    ap.add_argument("--experts", type=int, default=wl.C5.E,
                    help="number of routed experts (fewer than 256 keeps the weights small enough for a profiler capture)")
    ap.add_argument("--fp8", action="store_true", help="the FP8 (E4M3) precision variant instead of bf16")
    ap.add_argument("--zipf", type=float, default=wl.C5.zipf_s,
                    help="exponent of the expert popularity (0 = uniform routing with a selection bias, as in workloads C2/C4)")
    ap.add_argument("--route-only", action="store_true", help="time stage a1 (routing) by itself; no weights are allocated")
    args = ap.parse_args()
    B.load_library()
    hbm, tfl, src = load_peaks()
    if args.route_only:
        route_only(args.tokens, args.experts, wl.C5.k, args.zipf, hbm, src)
        return
    import dataclasses
    base = dataclasses.replace(wl.C5, E=args.experts, zipf_s=args.zipf, select_bias=args.zipf == 0)
    weights = (wl.make_weights_fp8 if args.fp8 else wl.make_weights)(base, 2, "cuda")
    for T in args.tokens:
        shape = base.with_tokens(T)
        step_us, n, stages, counts = run_one(shape, weights, args.iters_min_ms, fp8=args.fp8)
        floor_us, fl_us, by_us = layer_floor_us(shape, counts, hbm, tfl, fp8=args.fp8)
        cf = counts.double()
        nz = int((counts > 0).sum())
        print(json.dumps({
            "workload": f"C5 zipf(1.2) E={shape.E} T={T}" + (" fp8" if args.fp8 else ""), "phase": "decode" if T <= 256 else "prefill", "iters": n,
            "step_us": round(step_us, 1), "tokens_per_s": round(T / (step_us * 1e-6), 1),
            "roofline_floor_us": round(floor_us, 1), "frac_of_roofline": round(floor_us / step_us, 3),
            "floor_tensor_only_us": round(fl_us, 1), "floor_bytes_only_us": round(by_us, 1),
            "peaks": {"hbm_gbs": hbm, "bf16_tflops": tfl, "source": src},
            "imbalance_max_over_mean": round(float(cf.max() * shape.E / cf.sum()), 2),
            "cv": round(float(cf.std(unbiased=False) / cf.mean()), 2), "nonempty_experts": nz,
            "max_rows_per_expert": int(counts.max()), "stages_us": stages}), flush=True)


if __name__ == "__main__":
    main()
