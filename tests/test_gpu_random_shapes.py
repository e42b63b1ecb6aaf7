"""Whole layer against the oracle on a fixed list of randomly drawn shapes: odd token counts, expert counts
that are not multiples of 32, every k up to 8, H and I any multiple of 64, with and without a shared expert,
skewed and uniform routing, each GEMM variant, the row gather and a segmented FFN.  The list is drawn from a
seeded generator, so every run tests the same cases."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_layer_strict, layer_errors, np_f32, np_i32
from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _draw_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        E = int(rng.choice([2, 3, 5, 8, 17, 33, 40, 64, 96, 130]))
        k = int(rng.integers(1, min(E, 8) + 1))
        H = 64 * int(rng.integers(1, 9))
        I = 64 * int(rng.integers(1, 7))
        shared_I = 64 * int(rng.integers(1, 4)) if rng.random() < 0.4 else 0
        # prefill-sized (hundreds to a few thousand rows, several tiles and a ragged tail) or decode-sized
        T = int(rng.integers(130, 1200)) if i % 2 == 0 else int(rng.integers(1, 130))
        mode = ["auto", "large", "small", "gather", "segments"][i % 5]
        cases.append((i, T, H, E, k, I, shared_I, bool(rng.random() < 0.5), mode))
    return cases


CASES = _draw_cases(30, 20260993)


def _weights(shape, seed):
    w = wl.make_weights(shape, seed, DEV)
    for n in ("w_gate_up", "w_down", "ws_gate_up", "ws_down"):
        if w[n] is not None:  # unit-variance pre-activations, so that errors are visible against the tolerance
            w[n] = (w[n].float() * (1.0 / (0.02 * (w[n].shape[-1] ** 0.5)))).to(torch.bfloat16)
    return w


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"{c[0]}-T{c[1]}-H{c[2]}-E{c[3]}-k{c[4]}-I{c[5]}-S{c[6]}-{c[8]}")
def test_random_shape(case):
    i, T, H, E, k, I, shared_I, skew, mode = case
    shape = wl.LayerShape("r", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    w, a = _weights(shape, 700 + i), wl.make_activations(shape, 800 + i, DEV)
    if skew:  # Zipf-like popularity: a few hot experts, some experts empty
        a["logits"] = (a["logits"] + wl.zipf_log_weight(E, 1.2, 900 + i, DEV)).contiguous()
    phase = B.MOE_PHASE_PREFILL if T >= 130 else B.MOE_PHASE_DECODE
    variant = {"large": B.MOE_GEMM_LARGE_M, "small": B.MOE_GEMM_SMALL_M}.get(mode, B.MOE_GEMM_AUTO)
    gather = 1 if mode == "gather" else 0
    if gather:
        phase = B.MOE_PHASE_PREFILL
    ctx = B.MoeContext(B.make_config(H, E, k, I, shared_I, T, phase, 0, variant, row_gather=gather))
    if mode == "segments":
        ctx.moe_ctx_set_segments(max(1, E // 3))
    torch.cuda.synchronize()
    out, bufs = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    ref = oracle.layer(wl.bits(a["x"]), np_f32(a["logits"]), np_f32(a["bias"]), k, wl.bits(w["w_gate_up"]),
                       wl.bits(w["w_down"]), None if shared_I == 0 else wl.bits(w["ws_gate_up"]),
                       None if shared_I == 0 else wl.bits(w["ws_down"]))
    for name in ("topk_idx", "counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(np_i32(bufs[name]).reshape(-1), np.asarray(ref[name]).reshape(-1)), name
    check_layer_strict(out, ref, label=f"case {i}")
    ctx.close()


@pytest.mark.parametrize("case", CASES[:15], ids=lambda c: f"fp8-{c[0]}-T{c[1]}-H{c[2]}-E{c[3]}-k{c[4]}-I{c[5]}-S{c[6]}-{c[8]}")
def test_random_shape_fp8(case):
    """The FP8 (E4M3) precision variant on the same list, against the oracle's statement of its recipe."""
    i, T, H, E, k, I, shared_I, skew, mode = case
    shape = wl.LayerShape("r8", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    w8 = wl.make_weights_fp8(shape, 700 + i, DEV, std=1.0)
    for name, fan in (("sw_gate_up", H), ("sws_gate_up", H), ("sw_down", I), ("sws_down", shared_I)):
        if w8[name] is not None:
            w8[name] = (w8[name] / fan ** 0.5).contiguous()
    a = wl.make_activations(shape, 800 + i, DEV)
    if skew:
        a["logits"] = (a["logits"] + wl.zipf_log_weight(E, 1.2, 900 + i, DEV)).contiguous()
    phase = B.MOE_PHASE_PREFILL if T >= 130 else B.MOE_PHASE_DECODE
    variant = {"large": B.MOE_GEMM_LARGE_M, "small": B.MOE_GEMM_SMALL_M}.get(mode, B.MOE_GEMM_AUTO)
    ctx = B.MoeContext(B.make_config(H, E, k, I, shared_I, T, phase, 0, variant, weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    if mode == "segments":
        ctx.moe_ctx_set_segments(max(1, E // 3))
    torch.cuda.synchronize()
    out, bufs = ctx.layer_fp8(a["x"], a["logits"], a["bias"], w8)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    h = {n: (None if v is None else v.cpu().numpy()) for n, v in w8.items()}
    ref = oracle.layer_fp8(wl.bits(a["x"]), np_f32(a["logits"]), np_f32(a["bias"]), k, h["wq_gate_up"], h["sw_gate_up"],
                           h["wq_down"], h["sw_down"], h["wsq_gate_up"], h["sws_gate_up"], h["wsq_down"], h["sws_down"])
    for name in ("topk_idx", "counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(np_i32(bufs[name]).reshape(-1), np.asarray(ref[name]).reshape(-1)), name
    e = layer_errors(out, ref["out"])
    assert e["rel_l2"] <= 5e-3, e
    ctx.close()
