"""Degenerate and ragged cases of the whole layer against the oracle: empty batch, single token, k = 1, k = E,
one expert, the smallest dimensions, a context reused with shrinking and growing T, a caller's own routing
with repeated experts, a non-unit routed scale, and the host-buffer entry point on a decode context."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_layer_strict, layer_errors, np_f32, np_i32
from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
PHASES = [(B.MOE_PHASE_PREFILL, "P"), (B.MOE_PHASE_DECODE, "D")]


def _scaled_weights(shape, seed):
    w = wl.make_weights(shape, seed, DEV)
    for n in ("w_gate_up", "w_down", "ws_gate_up", "ws_down"):
        if w[n] is not None:
            w[n] = (w[n].float() * (1.0 / (0.02 * (w[n].shape[-1] ** 0.5)))).to(torch.bfloat16)
    return w


def _oracle(a, w, k, scale=1.0):
    return oracle.layer(wl.bits(a["x"]), np_f32(a["logits"]), None if a["bias"] is None else np_f32(a["bias"]), k,
                        wl.bits(w["w_gate_up"]), wl.bits(w["w_down"]),
                        None if w["ws_gate_up"] is None else wl.bits(w["ws_gate_up"]),
                        None if w["ws_down"] is None else wl.bits(w["ws_down"]), routed_scale=scale)


def _check(out, ref, label, term_abs=None):
    """ref: the staged oracle's result dict, or an output array with its term magnitude."""
    if isinstance(ref, dict):
        return check_layer_strict(out, ref, label)
    e = layer_errors(out, ref)
    assert e["rel_l2"] <= 5e-3 and e["worst_token_rel_l2"] <= 1e-2, f"{label}: {e}"
    assert e["max_abs"] <= 2.0 ** -7 * (float(np.max(term_abs)) + 1e-3), f"{label}: {e}"


@pytest.mark.parametrize("phase,pname", PHASES)
@pytest.mark.parametrize("T,H,E,k,I,shared_I", [
    (1, 256, 8, 2, 128, 0),      # a single token
    (1, 512, 16, 4, 256, 128),   # a single token with a shared expert
    (40, 64, 4, 1, 64, 0),       # k = 1 and the smallest H and I
    (40, 128, 4, 4, 64, 64),     # k = E: every expert takes every token
    (300, 128, 1, 1, 192, 0),    # a single expert: the layer is a dense MLP
    (129, 192, 3, 2, 320, 64),   # one row past a tile boundary; H, I not powers of two
    (200, 2560, 512, 8, 256, 0), # the paper's model shape: hidden 2,560, 512 routed experts, top-8 (I is not stated there)
    (70, 128, 1024, 32, 64, 0),  # the largest E and k the library accepts (single-CTA layout)
    (600, 128, 1024, 32, 64, 64),  # the same with 19200 routed rows: the multi-CTA layout with E = 1024
])
def test_small_and_degenerate_shapes(phase, pname, T, H, E, k, I, shared_I):
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    w, a = _scaled_weights(shape, 41), wl.make_activations(shape, 42, DEV)
    ctx = B.MoeContext(B.make_config(H, E, k, I, shared_I, T, phase))
    torch.cuda.synchronize()
    out, bufs = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    ref = _oracle(a, w, k)
    assert np.array_equal(np_i32(bufs["topk_idx"]), ref["topk_idx"])
    assert np.array_equal(np_i32(bufs["perm"]), ref["perm"])
    _check(out, ref, f"{pname} T={T} E={E} k={k}")
    ctx.close()


@pytest.mark.parametrize("phase,pname", PHASES)
def test_empty_batch_is_a_no_op(phase, pname):
    shape = wl.LayerShape("t", T=8, H=128, E=4, k=2, I=64, shared_I=64)
    w, a = _scaled_weights(shape, 1), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(128, 4, 2, 64, 64, 8, phase))
    bufs = B.alloc_step_buffers(0, 2, 4, DEV)
    bufs["counts"].fill_(-1); bufs["offsets"].fill_(-1)
    out = torch.full((8, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    ctx.moe_route(a["logits"][:0], None, bufs["topk_idx"], bufs["topk_w"], T=0)
    ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"][:0], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"], T=0)
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"][:0], w["ws_gate_up"], w["ws_down"], T=0)
    ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out[:0], T=0)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    assert torch.all(bufs["counts"] == 0) and torch.all(bufs["offsets"] == 0)
    assert torch.all(out == 7.0)
    # and the context still works afterwards
    o2, _ = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    _check(o2, _oracle(a, w, 2), f"{pname} after empty")
    ctx.close()


def test_context_reused_with_varying_token_counts():
    """Eager variable-length prefill: T changes on every call; stale rows from a larger batch never leak."""
    shape = wl.LayerShape("t", T=700, H=256, E=8, k=2, I=128, shared_I=64)
    w = _scaled_weights(shape, 5)
    ctx = B.MoeContext(B.make_config(256, 8, 2, 128, 64, 700, B.MOE_PHASE_PREFILL))
    for i, T in enumerate((700, 3, 257, 128, 699, 1)):
        a = wl.make_activations(shape.with_tokens(T), 50 + i, DEV)
        torch.cuda.synchronize()
        out, _ = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
        torch.cuda.synchronize()
        _check(out, _oracle(a, w, 2), f"T={T}")
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.close()


def test_callers_own_routing_with_repeated_experts_and_scale():
    """moe_route is optional: the caller may route itself, even sending a token to the same expert twice."""
    T, H, E, k, I = 96, 256, 6, 3, 128
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=I)
    w, a = _scaled_weights(shape, 7), wl.make_activations(shape, 8, DEV)
    g = torch.Generator(device=DEV).manual_seed(9)
    idx = torch.randint(0, E, (T, k), generator=g, device=DEV, dtype=torch.int32)  # repeats are likely
    wts = torch.rand(T, k, generator=g, device=DEV) * 0.7
    ctx = B.MoeContext(B.make_config(H, E, k, I, 0, T, B.MOE_PHASE_PREFILL))
    bufs = B.alloc_step_buffers(T, k, E, DEV)
    out = torch.empty(T, H, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    ctx.moe_dispatch_layout(idx, a["x"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"])
    ctx.moe_combine(wts, bufs["inv_perm"], out)
    torch.cuda.synchronize()
    counts, offsets, perm, inv = oracle.layout(np_i32(idx).reshape(-1), E)
    assert np.array_equal(np_i32(bufs["perm"]), perm)
    ref, mag = oracle.layer_tokens(wl.bits(a["x"]), np_i32(idx), np_f32(wts), wl.bits(w["w_gate_up"]),
                                   wl.bits(w["w_down"]), want_term_abs=True)
    _check(out, ref, "own routing", term_abs=mag)
    # routed_scale multiplies the routed weights
    ctx2 = B.MoeContext(B.make_config(H, E, k, I, 0, T, B.MOE_PHASE_PREFILL, routed_scale=2.5))
    o2, b2 = ctx2.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    torch.cuda.synchronize()
    assert abs(np_f32(b2["topk_w"]).sum(1) - 2.5).max() < 1e-5
    _check(o2, _oracle(a, w, k, scale=2.5), "routed_scale")
    ctx.close(); ctx2.close()


def test_host_buffer_entry_point_on_a_decode_context():
    shape = wl.LayerShape("t", T=24, H=512, E=16, k=4, I=256, shared_I=128, select_bias=True)
    w, a = _scaled_weights(shape, 11), wl.make_activations(shape, 12, DEV)
    ctx = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 32, B.MOE_PHASE_DECODE))
    out_h = torch.empty(24, 512, dtype=torch.bfloat16).pin_memory()
    for _ in range(2):  # both buffer sets
        out_h.zero_()
        ctx.moe_layer_host(a["logits"].cpu().pin_memory(), a["bias"], a["x"].cpu().pin_memory(), w["w_gate_up"],
                           w["w_down"], w["ws_gate_up"], w["ws_down"], out_h)
        _check(out_h, _oracle(a, w, 4), "host entry point")
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.close()
