#!/usr/bin/env python
"""Benchmark of the MoE-layer hot path (route -> dispatch layout -> grouped SwiGLU FFN -> combine).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-pd]

A step is one pass of the whole hot path over one batch of synthetic tokens.  The headline workload is
the prefill layer (Qwen3-30B-A3B-shaped, T=8192): `value` = prefill tokens/s with inputs resident in HBM,
`e2e` = the same through the host-buffer entry point (pinned host -> device -> host inside the timed
region).  The decode half of the metric (decode-step latency p50/p99 alone and under concurrent prefill,
DeepSeek-V3-shaped layer, two phase contexts on two streams) is reported under "decode".

With N > 1 (launched by torchrun, one rank per GPU) every rank runs its own batch against its own
replica of the weights -- tokens are independent, so there is no data-path collective; torch.distributed
is used only for the barrier and the max-over-ranks of the device time ("scaling": "weak").

`--impl reference` times the CPU oracle (the plain definition in oracle/) on a bounded sample of the same
workload on the host cores; it is a deliberately slow program, reported as context.
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

METRIC = "moe_layer_prefill_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu capture
# summarised in profiles/ (None until a capture of this workload exists).
DOMINANT_KERNEL_DRAM_BYTES = 1.0776e9 + 95.7e6  # profiles/grouped_gemm_tc_C3_prefill.md, GEMM1 + SwiGLU on C3


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons every 10 ms through NVML while the timed
    regions run; read-only.  Falls back to polling nvidia-smi if NVML cannot be loaded."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._how = None

    def _nvml_loop(self, nv, handle):
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(handle))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def _smi_loop(self):
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                stderr=subprocess.DEVNULL, text=True)
        self._proc = proc
        for ln in proc.stdout:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                self.samples.append(float(parts[0]))
                self.max_mhz = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    self.reasons.add(n)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            # NVML orders devices by PCI bus id; honour CUDA_VISIBLE_DEVICES when it is a plain index list
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.index
            if vis and all(v.strip().isdigit() for v in vis.split(",")):
                idx = int(vis.split(",")[self.index])
            handle = nv.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self._how = "nvml"
        except Exception:
            self._thread = threading.Thread(target=self._smi_loop, daemon=True)
            self._how = "nvidia-smi"
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._how == "nvidia-smi" and getattr(self, "_proc", None) is not None:
            time.sleep(0.1)
            self._proc.terminate()
        if self._thread is not None:
            self._thread.join(timeout=2)
        sm = self.samples
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": self.max_mhz,
                "sm_min_mhz": min(sm) if sm else None, "reasons": sorted(self.reasons), "samples": len(sm),
                "source": self._how}


# ------------------------------------------------------------------------------------------------ oracle arm

def oracle_inputs(shape, n_tokens, seed=3):
    """Host inputs for the oracle: the workload's layer with the first n_tokens tokens."""
    from paper_2609_00993_b200 import workloads as wl
    sub = shape.with_tokens(n_tokens)
    w = wl.make_weights(sub, seed, "cpu")
    a = wl.make_activations(sub, seed, "cpu")
    return (wl.bits(a["x"]), a["logits"].numpy(), None if a["bias"] is None else a["bias"].numpy(), sub.k,
            wl.bits(w["w_gate_up"]), wl.bits(w["w_down"]),
            None if w["ws_gate_up"] is None else wl.bits(w["ws_gate_up"]),
            None if w["ws_down"] is None else wl.bits(w["ws_down"]))


def oracle_sample_rate(oargs):
    """Times the oracle (all stages a1..a9, as it stands) on prepared inputs; (tokens/s, seconds, threads)."""
    import oracle
    oracle.route(oargs[1][:1], None, oargs[3])  # load the library outside the timed span
    t0 = time.perf_counter()
    oracle.layer(*oargs)
    dt = time.perf_counter() - t0
    return oargs[0].shape[0] / dt, dt, oracle.num_threads()


def run_reference(args):
    from paper_2609_00993_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shape = wl.C3
    n = args.ref_step_tokens
    oargs = oracle_inputs(shape, n)
    times, cores = [], 1
    for i in range(args.warmup + args.steps):
        r, dt, cores = oracle_sample_rate(oargs)
        if i >= args.warmup:
            times.append(dt)
    value = n * len(times) / sum(times)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(shape), "sample": f"first {n} tokens per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"all stages on the first {n} of {shape.T} tokens, per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def workload_name(shape):
    return (f"{shape.name}: T={shape.T} H={shape.H} E={shape.E} top-{shape.k} I={shape.I} "
            f"shared_I={shape.shared_I} bf16, fp32 router logits")


# --------------------------------------------------------------------------------------------------- our arm

def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's figure (all ranks get it); with one process it is the value itself."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / seconds


def percentile(vals, q):
    import numpy as np
    return float(np.percentile(np.asarray(vals, dtype=np.float64), q))


def decode_under_prefill(torch, B, wl, dev, iters, warm):
    """Config 4: D steps (T=64) on stream D alone, with an idle P context, serial with P, and while P batches
    (T=4096) run back to back on stream P.  Each phase has its own context; weights are shared read-only."""
    w = wl.make_weights(wl.C2, 2, dev)
    sp, sd = torch.cuda.Stream(device=dev, priority=0), torch.cuda.Stream(device=dev, priority=-1)
    n_in = 4  # rotating input sets (fresh seeds), generated before the timed regions
    aps = [wl.make_activations(wl.C4_P, 4000 + i, dev) for i in range(n_in)]
    ads = [wl.make_activations(wl.C4_D, 5000 + i, dev) for i in range(n_in)]
    mk = lambda s, ph, st: B.MoeContext(B.make_config(s.H, s.E, s.k, s.I, s.shared_I, s.T, ph), stream=st, device=dev)
    ctx_d = mk(wl.C4_D, B.MOE_PHASE_DECODE, sd)
    bd = B.alloc_step_buffers(wl.C4_D.T, 8, 256, dev)
    od = torch.empty(wl.C4_D.T, 7168, dtype=torch.bfloat16, device=dev)
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])

    def d_step(i):
        a = ads[i % n_in]
        ctx_d.layer(a["x"], a["logits"], a["bias"], *wargs, out=od, bufs=bd)

    def time_d(n, before=None):
        evs = []
        for i in range(n):
            if before:
                before(i)
            with torch.cuda.stream(sd):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(sd); d_step(i); e1.record(sd)
            evs.append((e0, e1))
        torch.cuda.synchronize(dev)
        return [1e3 * e0.elapsed_time(e1) for e0, e1 in evs]  # microseconds

    res = {}
    torch.cuda.synchronize(dev)
    time_d(warm)
    alone = time_d(iters)
    res["alone_us"] = {"p50": percentile(alone, 50), "p99": percentile(alone, 99), "max": max(alone)}
    # the same step as the host sees it: from the first enqueue to the end of a stream synchronisation
    wall = []
    for i in range(max(20, iters // 4)):
        t0 = time.perf_counter()
        with torch.cuda.stream(sd):
            d_step(i)
        sd.synchronize()
        wall.append(1e6 * (time.perf_counter() - t0))
    res["alone_host_wall_us"] = {"p50": percentile(wall, 50), "p99": percentile(wall, 99)}

    # the same D step replayed from a CUDA graph (stable phase-owned addresses): launch overhead off the path
    try:
        graph = torch.cuda.CUDAGraph()
        a0 = ads[0]
        with torch.cuda.graph(graph, stream=sd):
            ctx_d.layer(a0["x"], a0["logits"], a0["bias"], *wargs, out=od, bufs=bd)
        evs = []
        for _ in range(iters):
            with torch.cuda.stream(sd):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(sd); graph.replay(); e1.record(sd)
            evs.append((e0, e1))
        torch.cuda.synchronize(dev)
        rep = [1e3 * a.elapsed_time(b) for a, b in evs]
        res["graph_replay_us"] = {"p50": percentile(rep, 50), "p99": percentile(rep, 99)}
        del graph
    except Exception as exc:
        res["graph_replay_us"] = {"error": repr(exc)}

    # the same D step with FP8 weights (half the weight bytes to stream)
    try:
        w8 = wl.make_weights_fp8(wl.C2, 2, dev)
        torch.cuda.synchronize(dev)  # the weights are generated on torch's current stream, the steps run on sd
        s = wl.C4_D
        ctx_d8 = B.MoeContext(B.make_config(s.H, s.E, s.k, s.I, s.shared_I, s.T, B.MOE_PHASE_DECODE,
                                            weight_format=B.MOE_WEIGHTS_FP8_E4M3), stream=sd, device=dev)
        evs = []
        for i in range(warm + iters):
            a = ads[i % n_in]
            with torch.cuda.stream(sd):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(sd); ctx_d8.layer_fp8(a["x"], a["logits"], a["bias"], w8, out=od, bufs=bd); e1.record(sd)
            evs.append((e0, e1))
        torch.cuda.synchronize(dev)
        t8 = [1e3 * a.elapsed_time(b) for a, b in evs[warm:]]
        res["fp8_alone_us"] = {"p50": percentile(t8, 50), "p99": percentile(t8, 99),
                               "device_status": ctx_d8.moe_ctx_status()}
        ctx_d8.close()
        del w8
        torch.cuda.empty_cache()
    except Exception as exc:
        res["fp8_alone_us"] = {"error": repr(exc)}

    ctx_p = mk(wl.C4_P, B.MOE_PHASE_PREFILL, sp)
    bp = B.alloc_step_buffers(wl.C4_P.T, 8, 256, dev)
    op = torch.empty(wl.C4_P.T, 7168, dtype=torch.bfloat16, device=dev)

    def p_step(i):
        a = aps[i % n_in]
        ctx_p.layer(a["x"], a["logits"], a["bias"], *wargs, out=op, bufs=bp)

    idle = time_d(iters)
    res["with_idle_p_context_us"] = {"p50": percentile(idle, 50), "p99": percentile(idle, 99)}

    # P alone
    for i in range(3):
        p_step(i)
    torch.cuda.synchronize(dev)
    n_p = max(8, iters // 10)
    with torch.cuda.stream(sp):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(sp)
        for i in range(n_p):
            p_step(i)
        e1.record(sp)
    torch.cuda.synchronize(dev)
    p_alone_ms = e0.elapsed_time(e1) / n_p
    res["prefill_alone_tokens_per_s"] = wl.C4_P.T / (p_alone_ms * 1e-3)

    # (1) concurrent, no segmentation: stream P kept saturated with whole P batches, D steps timed one by one;
    #     only the stream priority separates the phases
    inflight = []

    def feed_p(i):
        # at most two P batches queued ahead, so that P is always in flight but the queue stays short
        while len(inflight) >= 2:
            inflight.pop(0).synchronize()
        p_step(i)
        ev = torch.cuda.Event()
        ev.record(sp)
        inflight.append(ev)

    n_unseg = max(20, iters // 4)
    with torch.cuda.stream(sp):
        pe0 = torch.cuda.Event(enable_timing=True); pe0.record(sp)
    conc = time_d(n_unseg, before=feed_p)
    with torch.cuda.stream(sp):
        pe1 = torch.cuda.Event(enable_timing=True); pe1.record(sp)
    torch.cuda.synchronize(dev)
    res["concurrent_unsegmented_us"] = {"p50": percentile(conc, 50), "p99": percentile(conc, 99), "max": max(conc),
                                        "prefill_tokens_per_s": wl.C4_P.T * n_unseg / (pe0.elapsed_time(pe1) * 1e-3)}
    inflight.clear()

    # (2) segment turnstile: P is cut at safe boundaries (one launch per `span` experts); the host controller
    #     admits the waiting D step at the first boundary after it became ready and holds P's next segment
    #     until that D step is done.  Per iteration one P batch and one D step, as in config 4.
    #     Arrival model (worst case per step): the D batch becomes ready the moment a randomly chosen P
    #     segment b starts executing, so it waits for the whole of segment b and is admitted at the boundary
    #     after it.  The start event of the D step is therefore ordered after segment b-1, its kernels after
    #     segment b, and P's segment b+1 after the D step.
    import random

    def turnstile_run(span, n_iter, seed=0):
        rng = random.Random(seed)
        st = {"target": 0, "i": 0, "prev": None, "evs": []}

        def at_boundary(b, nb):
            after_b = torch.cuda.Event()
            after_b.record(sp)
            if b == st["target"] % nb:
                with torch.cuda.stream(sd):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    sd.wait_event(st["prev"])   # D becomes ready as segment b starts
                    e0.record(sd)
                    sd.wait_event(after_b)      # ... and is admitted at the boundary after it
                    d_step(st["i"])
                    e1.record(sd)
                sp.wait_event(e1)               # P's next segment is released after the D step
                st["evs"].append((e0, e1))
            st["prev"] = after_b

        ctx_p.moe_ctx_set_segments(span, at_boundary)
        torch.cuda.synchronize(dev)
        with torch.cuda.stream(sp):
            t0 = torch.cuda.Event(enable_timing=True); t0.record(sp)
        for i in range(n_iter):
            st["target"], st["i"] = rng.randrange(1 << 20), i
            start = torch.cuda.Event()
            start.record(sp)
            st["prev"] = start
            p_step(i)
            if i % 4 == 3:
                torch.cuda.synchronize(dev)  # keep the host at most a few batches ahead of the device
        with torch.cuda.stream(sp):
            t1 = torch.cuda.Event(enable_timing=True); t1.record(sp)
        torch.cuda.synchronize(dev)
        ctx_p.moe_ctx_set_segments(0)
        us = [1e3 * a.elapsed_time(b) for a, b in st["evs"]]
        return {"span_experts": span, "d_steps": len(us), "p50": percentile(us, 50), "p99": percentile(us, 99),
                "max": max(us), "prefill_tokens_per_s": wl.C4_P.T * n_iter / (t0.elapsed_time(t1) * 1e-3),
                "p99_over_alone": percentile(us, 99) / res["alone_us"]["p99"]}

    turnstile_run(16, 8)  # warm-up
    res["turnstile"] = [turnstile_run(span, iters if span == 16 else max(20, iters // 4)) for span in (8, 16, 32, 64)]
    best = [r for r in res["turnstile"] if r["span_experts"] == 16][0]
    res["concurrent_us"] = {"p50": best["p50"], "p99": best["p99"], "max": best["max"],
                            "policy": "segment turnstile, 16 experts per P segment"}
    res["prefill_concurrent_tokens_per_s"] = best["prefill_tokens_per_s"]
    res["p99_ratio_concurrent_over_alone"] = best["p99_over_alone"]

    # (3) serial: the D batch becomes ready as a whole (unsegmented) P batch starts and waits for all of it
    ser = []
    for i in range(max(8, iters // 10)):
        start = torch.cuda.Event()
        start.record(sp)
        p_step(i)
        with torch.cuda.stream(sd):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            sd.wait_event(start)
            e0.record(sd)
            sd.wait_stream(sp)
            d_step(i)
            e1.record(sd)
        sp.wait_stream(sd)
        ser.append((e0, e1))
    torch.cuda.synchronize(dev)
    ser_us = [1e3 * a.elapsed_time(b) for a, b in ser]
    res["serial_us"] = {"p50": percentile(ser_us, 50), "p99": percentile(ser_us, 99),
                        "note": "D ready at the start of an unsegmented P batch, runs after it"}
    res["prefill_serial_tokens_per_s"] = wl.C4_P.T / ((p_alone_ms + res["alone_us"]["p50"] * 1e-3) * 1e-3)
    # how much of a P batch plus one D step the turnstile run hides by running them at the same time: 0 % means
    # strict time slicing (the turnstile admits D between P segments and P waits for it), 100 % would hide all of D,
    # a negative figure means that cutting P into segments costs more than is hidden
    t_p, t_d = p_alone_ms * 1e-3, res["alone_us"]["p50"] * 1e-6
    t_conc = wl.C4_P.T / res["prefill_concurrent_tokens_per_s"]  # seconds per P batch while D steps run
    res["overlap_pct"] = 100.0 * (t_p + t_d - t_conc) / t_d
    res["iterations"] = iters
    res["workload"] = "C4: P T=4096 on stream P || D T=64 on stream D (high priority), DeepSeek-V3-shaped layer"
    ctx_p.close(); ctx_d.close()
    del w
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    from paper_2609_00993_b200 import binding as B
    from paper_2609_00993_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback of the product path")
    B.load_library()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    shape = wl.C3
    T, H, E, k, I = shape.T, shape.H, shape.E, shape.k, shape.I
    w = wl.make_weights(shape, 3 + rank, dev)
    n_in = 4  # rotate through several input batches; weights (1.2 GB) + activations exceed L2 every step
    acts = [wl.make_activations(shape, 300 + 16 * rank + i, dev) for i in range(n_in)]
    stream = torch.cuda.Stream(device=dev)
    ctx = B.MoeContext(B.make_config(H, E, k, I, shape.shared_I, T, B.MOE_PHASE_PREFILL), stream=stream, device=dev)
    bufs = B.alloc_step_buffers(T, k, E, dev)
    out = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])

    def step(i):
        a = acts[i % n_in]
        ctx.layer(a["x"], a["logits"], a["bias"], *wargs, out=out, bufs=bufs)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(n, fn):
        barrier()
        with torch.cuda.stream(stream):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(n):
                fn(i)
            e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev)

    torch.cuda.synchronize(dev)
    for i in range(args.warmup):
        with torch.cuda.stream(stream):
            step(i)
    torch.cuda.synchronize(dev)
    assert ctx.moe_ctx_status() == B.MOE_OK

    # ---- device-resident timed region (exactly K steps)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    l0 = ctx.moe_ctx_launch_count()
    ms_total = timed(args.steps, step)
    launches = ctx.moe_ctx_launch_count() - l0
    ms_per_step = ms_total / args.steps
    value = whole_job_rate(T, world, ms_per_step * 1e-3)

    # ---- the same K steps again with per-kernel events, for the roofline of the dominant kernel
    ctx.moe_ctx_set_profiling(True)
    timed(args.steps, step)
    prof = ctx.moe_ctx_read_profile()
    ctx.moe_ctx_set_profiling(False)
    clocks = sampler.stop() if rank == 0 else None  # sampled over the timed region and its per-kernel repeat
    stage_us = {n: (1e3 * ms / c if c else None) for n, (ms, c) in prof.items()}

    # ---- launch floor: the library's smallest launch (the T = 0 layout: one 256-thread CTA that clears E + 1 words),
    # 100 of them back to back replayed from a CUDA graph, so that the host's call overhead is off the path: the
    # device time a dependent kernel costs before it does any work
    n_floor = 100
    launch_floor_us = None
    try:
        floor_graph = torch.cuda.CUDAGraph()
        # thread-local capture mode: other threads of the process (a process group's watchdog) may keep calling CUDA
        with torch.cuda.graph(floor_graph, stream=stream, capture_error_mode="thread_local"):
            for _ in range(n_floor):
                ctx.moe_dispatch_layout(bufs["topk_idx"], None, T=0)
                ctx.moe_ctx_abandon_step()
        floor_graph.replay()
        launch_floor_us = 1e3 * timed(5, lambda i: floor_graph.replay()) / (5 * n_floor)
        del floor_graph
    except Exception:  # the figure is context for the layout time; the run goes on without it
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()

    # ---- variant: GEMM1 gathers its rows from x while it runs (no x_perm is written or re-read)
    fused = None
    if not args.quick:
        ctx_g = B.MoeContext(B.make_config(H, E, k, I, shape.shared_I, T, B.MOE_PHASE_PREFILL, row_gather=1),
                             stream=stream, device=dev)

        def step_g(i):
            a = acts[i % n_in]
            ctx_g.layer(a["x"], a["logits"], a["bias"], *wargs, out=out, bufs=bufs)

        with torch.cuda.stream(stream):
            for i in range(args.warmup):
                step_g(i)
        ms_g = timed(args.steps, step_g) / args.steps
        assert ctx_g.moe_ctx_status() == B.MOE_OK
        ctx_g.close()
        fused = {"ms_per_step": ms_g, "value": whole_job_rate(T, world, ms_g * 1e-3), "unit": UNIT,
                 "note": "row_gather=1: stage a5 fused into GEMM1 (cp.async row gather), x_perm not materialised"}

    # ---- precision variant: the same step with FP8 (E4M3) weights and on-the-fly per-row activation quantisation
    fp8 = None
    if not args.quick:
        w8 = wl.make_weights_fp8(shape, 3 + rank, dev)
        torch.cuda.synchronize(dev)
        ctx8 = B.MoeContext(B.make_config(H, E, k, I, shape.shared_I, T, B.MOE_PHASE_PREFILL,
                                          weight_format=B.MOE_WEIGHTS_FP8_E4M3), stream=stream, device=dev)

        def step8(i):
            a = acts[i % n_in]
            ctx8.layer_fp8(a["x"], a["logits"], a["bias"], w8, out=out, bufs=bufs)

        with torch.cuda.stream(stream):
            for i in range(args.warmup):
                step8(i)
        ms8 = timed(args.steps, step8) / args.steps
        ctx8.moe_ctx_set_profiling(True)
        timed(args.steps, step8)
        prof8 = ctx8.moe_ctx_read_profile()
        assert ctx8.moe_ctx_status() == B.MOE_OK
        ctx8.close()
        del w8
        us8 = {n: round(1e3 * ms / c, 1) for n, (ms, c) in prof8.items() if c}
        fp8 = {"ms_per_step": ms8, "value": whole_job_rate(T, world, ms8 * 1e-3), "unit": UNIT, "dtype": "e4m3",
               "stages_us": us8,
               "gemm1_TFLOPs": 4.0 * T * k * H * I / (us8["gemm1_swiglu"] * 1e-6) / 1e12,
               "note": "W8A8: E4M3 weights with per-output-channel scales, bf16 rows quantised per row on the fly, "
                       "tcgen05 kind::f8f6f4; not the headline (the metric is quoted on bf16)"}

    # ---- end to end: pinned host buffers in, pinned host buffer out, every copy inside the timed region.
    # Public API: moe_layer_host_submit / moe_layer_host_wait, four slots, so that the copies of one step overlap
    # the kernels of its neighbours; the synchronous moe_layer_host (copy, compute, copy, sync) is timed beside it.
    e2e_value = e2e_sync_value = None
    if not args.quick:
        hx = [a["x"].cpu().pin_memory() for a in acts]
        hl = [a["logits"].cpu().pin_memory() for a in acts]

        def host_step(i):
            ctx.moe_layer_host(hl[i % n_in], None, hx[i % n_in], *wargs, hout[0])

        n_slots = 4
        hout = [torch.empty(T, H, dtype=torch.bfloat16).pin_memory() for _ in range(n_slots)]

        def run_pipelined(n):
            for i in range(n):
                if i >= n_slots:
                    ctx.moe_layer_host_wait(i % n_slots)
                ctx.moe_layer_host_submit(i % n_slots, hl[i % n_in], None, hx[i % n_in], *wargs, hout[i % n_slots])
            for sl in range(n_slots):
                ctx.moe_layer_host_wait(sl)

        for i in range(max(3, args.warmup)):
            host_step(i)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.steps):
            host_step(i)
        torch.cuda.synchronize(dev)
        e2e_sync_value = whole_job_rate(T * args.steps, world, max_over_ranks(time.perf_counter() - t0, dist, dev))
        run_pipelined(max(4, args.warmup))
        barrier()
        t0 = time.perf_counter()
        run_pipelined(args.steps)
        torch.cuda.synchronize(dev)
        e2e_value = whole_job_rate(T * args.steps, world, max_over_ranks(time.perf_counter() - t0, dist, dev))
    assert ctx.moe_ctx_status() == B.MOE_OK

    if rank != 0:
        ctx.close()
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    peaks = load_peaks()
    N = T * k
    gemm1_flops = 4.0 * N * H * I            # gate and up projections: 2 * (2*N*H*I)
    gemm1_us = stage_us["gemm1_swiglu"]
    achieved = gemm1_flops / (gemm1_us * 1e-6) / 1e12
    # burst figure when the clocks stayed near maximum during the timed region, sustained figure otherwise
    burst = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and
                 clocks["sm_mhz"] >= 0.9 * clocks["sm_max_mhz"])
    peak = peaks["bf16_tflops"] if burst else peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    roofline = {"kernel": "grouped_gemm_stream_kernel<gated> (GEMM1 + SwiGLU, small-M variant)", "bound": "tensor",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": DOMINANT_KERNEL_DRAM_BYTES,
                "peak_source": f"of {peaks['_source']} ({'burst' if burst else 'sustained'} bf16 matmul)",
                "frac_of_sustained": achieved / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                "frac_of_nominal_2250": achieved / 2250.0,
                "flops_per_launch": gemm1_flops, "us_per_launch": gemm1_us,
                "algorithmic_bytes_per_launch": 2.0 * N * H + 2.0 * E * 2 * I * H + 2.0 * N * I}
    # per-stage achieved rates against the roofline that bounds each stage
    bw = peaks["hbm_gbs"]
    bytes_permute = 2.0 * T * H + 2.0 * N * H + 4.0 * N
    bytes_combine = 2.0 * N * H + 2.0 * T * H + 8.0 * N
    gemm2_flops = 2.0 * N * H * I
    # Bracketing every stage with its own pair of timing events drains the stream at each boundary, which the plain
    # timed region does not do: the sum of the bracketed stages exceeds the plain step by this much per stage
    # (the per-stage figures below are the bracketed, pessimistic ones).
    n_br = sum(1 for n in ("route", "layout", "permute", "gemm1_swiglu", "gemm2", "combine") if stage_us.get(n))
    bracket_overhead = (sum(stage_us[n] for n in ("route", "layout", "permute", "gemm1_swiglu", "gemm2", "combine")
                            if stage_us.get(n)) - 1e3 * ms_per_step) / max(n_br, 1)
    stages = {
        "event_bracket_overhead_us_per_stage": bracket_overhead,
        "route_us": stage_us["route"], "layout_us": stage_us["layout"],
        "layout": {"us": stage_us["layout"], "launches": 3, "launch_floor_us_per_launch": launch_floor_us,
                   "note": "counts + scan + placement move 1.3 MB at this size: three dependent launches of chained small loads, bound by latency, not by HBM"},
        "permute": {"us": stage_us["permute"], "GBps": bytes_permute / (stage_us["permute"] * 1e-6) / 1e9,
                    "frac_hbm": bytes_permute / (stage_us["permute"] * 1e-6) / 1e9 / bw},
        "gemm1_swiglu": {"us": gemm1_us, "TFLOPs": achieved, "frac_tensor": achieved / peak},
        "gemm2": {"us": stage_us["gemm2"], "TFLOPs": gemm2_flops / (stage_us["gemm2"] * 1e-6) / 1e12,
                  "frac_tensor": gemm2_flops / (stage_us["gemm2"] * 1e-6) / 1e12 / peak},
        "combine": {"us": stage_us["combine"], "GBps": bytes_combine / (stage_us["combine"] * 1e-6) / 1e9,
                    "frac_hbm": bytes_combine / (stage_us["combine"] * 1e-6) / 1e9 / bw},
    }

    # ---- CPU baseline: the oracle on a bounded sample, on this machine's host cores
    cpu_baseline = None
    if not args.quick:
        cpu_rate, cpu_dt, cores = oracle_sample_rate(oracle_inputs(shape, args.ref_tokens))
        cpu_baseline = {"value": cpu_rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"all stages on the first {args.ref_tokens} of {T} tokens ({cpu_dt:.1f} s)"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(shape), "phase": "prefill (small-M GEMM variant, chosen from 512 rows per expert)",
                       "l2": "inputs larger than L2: 1.2 GB of weights streamed per step, 4 rotating input batches",
                       "parallelism": f"replicas x{world} (no data-path collective)"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": T * E * 4 + T * H * 2,
                    "d2h_bytes_per_step": T * H * 2,
                    "api": "moe_layer_host_submit / moe_layer_host_wait, four slots in rotation (copies overlap kernels)",
                    "synchronous_moe_layer_host": e2e_sync_value},
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "stages": stages, "fused_row_gather": fused, "fp8_variant": fp8}
    ctx.close()
    del w, acts
    torch.cuda.empty_cache()
    if world == 1 and not args.no_pd and not args.quick:
        try:
            line["decode"] = decode_under_prefill(torch, B, wl, dev, args.pd_iters, 20)
        except Exception as exc:  # the headline number stands even if the P/D section cannot run
            line["decode"] = {"error": repr(exc)}
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--ref-tokens", type=int, default=8192, help="tokens of the cpu_baseline oracle sample")
    ap.add_argument("--ref-step-tokens", type=int, default=256, help="tokens per step of the reference (oracle) arm")
    ap.add_argument("--no-pd", action="store_true", help="skip the decode-under-prefill section")
    ap.add_argument("--quick", action="store_true",
                    help="device-resident timed region only (no e2e, cpu_baseline or decode section): the profiling case")
    ap.add_argument("--pd-iters", type=int, default=200)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
