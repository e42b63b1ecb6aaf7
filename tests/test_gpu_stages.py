"""Stage-by-stage parity of the CUDA path (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_topk_w, layer_errors, np_f32, np_i32
from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _ctx(H=256, E=8, k=2, I=512, shared_I=0, max_tokens=64, phase=B.MOE_PHASE_PREFILL, variant=B.MOE_GEMM_AUTO,
         sm_budget=0, row_gather=0):
    cfg = B.make_config(H, E, k, I, shared_I, max_tokens, phase, sm_budget, variant, row_gather=row_gather)
    return B.MoeContext(cfg)


# ------------------------------------------------------------------------------------------ a1 route

@pytest.mark.parametrize("T,E,k,bias", [
    (64, 8, 2, False),        # C1
    (128, 256, 8, True),      # C2 (vectorised key loads)
    (1000, 128, 8, False),    # C3 shape, ragged T
    (37, 512, 8, True),       # paper's model shape: top-8 of 512
    (5, 12, 12, False),       # k = E
    (9, 40, 1, True),         # k = 1
    (3, 1024, 32, False),     # the largest E and k
    (1, 256, 8, False),       # a single token
])
def test_route_matches_oracle(T, E, k, bias):
    g = torch.Generator(device=DEV).manual_seed(E * 7 + k)
    logits = torch.randn(T, E, generator=g, device=DEV)
    b = torch.randn(E, generator=g, device=DEV) * 0.5 if bias else None
    ctx = _ctx(E=E, k=k, max_tokens=T)
    idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    w = torch.empty(T, k, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    ctx.moe_route(logits, b, idx, w)
    torch.cuda.synchronize()
    ridx, rw = oracle.route(np_f32(logits), None if b is None else np_f32(b), k)
    assert np.array_equal(np_i32(idx), ridx)
    check_topk_w(w, rw)
    assert abs(np_f32(w).sum(1) - 1.0).max() <= 1e-6 * 4
    ctx.close()


@pytest.mark.parametrize("E,k", [(16, 4), (256, 8), (100, 7)])
def test_route_tie_rule(E, k):
    logits = wl.tie_heavy_logits(200, E, seed=E, device=DEV)
    ctx = _ctx(E=E, k=k, max_tokens=200)
    idx = torch.empty(200, k, dtype=torch.int32, device=DEV)
    w = torch.empty(200, k, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    ctx.moe_route(logits, None, idx, w)
    torch.cuda.synchronize()
    ridx, rw = oracle.route(np_f32(logits), None, k)
    assert np.array_equal(np_i32(idx), ridx)
    check_topk_w(w, rw)
    ctx.close()


def test_route_scale_and_all_equal():
    cfg = B.make_config(256, 16, 4, 512, 0, 8, routed_scale=2.5)
    ctx = B.MoeContext(cfg)
    logits = torch.full((8, 16), 0.75, device=DEV)
    idx = torch.empty(8, 4, dtype=torch.int32, device=DEV)
    w = torch.empty(8, 4, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    ctx.moe_route(logits, None, idx, w)
    torch.cuda.synchronize()
    assert np.array_equal(np_i32(idx), np.tile(np.arange(4, dtype=np.int32), (8, 1)))
    assert np.array_equal(np_f32(w), np.full((8, 4), 0.625, np.float32))
    ctx.close()


# ------------------------------------------------------------------------------- a2-a4 dispatch layout

@pytest.mark.parametrize("T,E,k", [
    (0, 8, 2),            # empty
    (1, 8, 2),
    (64, 8, 2),           # C1
    (128, 256, 8),        # C2: single-CTA path
    (2048, 256, 8),       # largest single-CTA case (16384 slots)
    (2049, 256, 8),       # first multi-CTA case, ragged last chunk
    (8192, 128, 8),       # C3
    (32768, 256, 8),      # C5 maximum
    (777, 1024, 3),       # largest E
    (513, 1, 1),          # one expert takes everything
])
def test_layout_matches_oracle(T, E, k):
    g = torch.Generator(device=DEV).manual_seed(T + E)
    # distinct experts per token, skewed popularity so that segments are uneven and some are empty
    pop = torch.rand(E, generator=g, device=DEV) ** 3 + 1e-4
    idx = (torch.multinomial(pop.expand(max(T, 1), E), k, replacement=False, generator=g)[:T]).to(torch.int32)
    ctx = _ctx(E=E, k=k, max_tokens=max(T, 1))
    bufs = B.alloc_step_buffers(T, k, E, DEV)
    torch.cuda.synchronize()
    ctx.moe_dispatch_layout(idx, None, bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"], T=T)
    torch.cuda.synchronize()
    counts, offsets, perm, inv = oracle.layout(np_i32(idx).reshape(-1), E)
    assert np.array_equal(np_i32(bufs["counts"]), counts)
    assert np.array_equal(np_i32(bufs["offsets"]), offsets)
    assert np.array_equal(np_i32(bufs["perm"]), perm)
    assert np.array_equal(np_i32(bufs["inv_perm"]), inv)
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.close()


@pytest.mark.parametrize("T", [16, 4000])
def test_layout_reports_bad_index_without_faulting(T):
    E, k = 8, 2
    g = torch.Generator(device=DEV).manual_seed(3)
    idx = torch.randint(0, E, (T, k), generator=g, device=DEV, dtype=torch.int32)
    idx[3, 1] = E + 5
    idx[T - 1, 0] = -2
    ctx = _ctx(E=E, k=k, max_tokens=T)
    bufs = B.alloc_step_buffers(T, k, E, DEV)
    torch.cuda.synchronize()
    ctx.moe_dispatch_layout(idx, None, bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"], T=T)
    assert ctx.moe_ctx_status() == B.MOE_ERR_BAD_INDEX
    assert ctx.moe_ctx_status() == B.MOE_OK  # reading clears it
    inv = np_i32(bufs["inv_perm"])
    assert inv[3 * k + 1] == -1 and inv[(T - 1) * k] == -1
    good = np_i32(idx).reshape(-1)
    keep = (good >= 0) & (good < E)
    assert np_i32(bufs["counts"]).sum() == keep.sum()
    # the surviving slots still form the stable layout of the valid indices
    order = np.argsort(good[keep], kind="stable")
    assert np.array_equal(np_i32(bufs["perm"])[:keep.sum()], np.nonzero(keep)[0][order])
    ctx.close()


# ------------------------------------------------------------------------------------------ a5 permute

@pytest.mark.parametrize("T,H,E,k", [(64, 256, 8, 2), (128, 7168, 256, 8), (1000, 2048, 128, 8), (3, 8192 + 64, 4, 4)])
def test_permute_is_bit_exact(T, H, E, k):
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=64)
    a = wl.make_activations(shape, 11, DEV)
    ctx = _ctx(H=H, E=E, k=k, I=64, max_tokens=T)
    bufs = B.alloc_step_buffers(T, k, E, DEV)
    torch.cuda.synchronize()
    ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])
    ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    torch.cuda.synchronize()
    xp = ctx.moe_ctx_debug_ptrs()["x_perm"][:T * k]
    ref = oracle.permute(wl.bits(a["x"]), np_i32(bufs["perm"]), k)
    assert np.array_equal(wl.bits(xp), ref)
    ctx.close()


# ------------------------------------------------------------------------------- a6-a8 FFN, a9 combine

def _run_step(ctx, a, w, T):
    bufs = B.alloc_step_buffers(T, ctx.cfg.top_k, ctx.cfg.n_experts, DEV)
    torch.cuda.synchronize()
    out, _ = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"],
                       bufs=bufs)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    return out, bufs


def _oracle_step(a, w, k, emulate=False):
    return oracle.layer(wl.bits(a["x"]), np_f32(a["logits"]), None if a["bias"] is None else np_f32(a["bias"]), k,
                        wl.bits(w["w_gate_up"]), wl.bits(w["w_down"]),
                        None if w["ws_gate_up"] is None else wl.bits(w["ws_gate_up"]),
                        None if w["ws_down"] is None else wl.bits(w["ws_down"]), emulate_bf16=emulate)


VARIANTS = [(B.MOE_GEMM_VALIDATION, B.MOE_PHASE_PREFILL, "validation", 0),
            (B.MOE_GEMM_LARGE_M, B.MOE_PHASE_PREFILL, "large-M", 0),
            (B.MOE_GEMM_LARGE_M, B.MOE_PHASE_PREFILL, "large-M-gather", 1),  # GEMM1 gathers its rows; no x_perm
            (B.MOE_GEMM_SMALL_M, B.MOE_PHASE_DECODE, "small-M", 0),
            (B.MOE_GEMM_SMALL_M, B.MOE_PHASE_PREFILL, "small-M-P", 0)]

SHAPES = [
    # T,   H,    E,  k, I,   shared_I
    (64, 256, 8, 2, 512, 0),       # C1
    (300, 512, 16, 4, 192, 128),   # several row tiles, ragged tails, I not a multiple of 128, shared expert
    (33, 1024, 64, 8, 128, 0),     # a few rows per expert; some experts empty
    (700, 320, 4, 2, 64, 64),      # H not a multiple of 128/256: partial feature tiles; K = 320 (5 k-blocks)
    (400, 512, 8, 4, 256, 128),    # ~200 rows per expert: tiles of 129..256 tokens
    (1100, 256, 3, 2, 128, 0),     # ~730 rows per expert: several token chunks per expert
]


@pytest.mark.parametrize("variant,phase,vname,row_gather", VARIANTS)
@pytest.mark.parametrize("T,H,E,k,I,shared_I", SHAPES)
def test_ffn_and_combine_match_oracle(variant, phase, vname, row_gather, T, H, E, k, I, shared_I):
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    w = wl.make_weights(shape, 5, DEV)
    # scale the weights up so that the outputs are O(1) and a wrong tile or a dropped k-block is far outside tolerance
    for n in ("w_gate_up", "w_down", "ws_gate_up", "ws_down"):
        if w[n] is not None:
            w[n] = (w[n].float() * (1.0 / (0.02 * (w[n].shape[-1] ** 0.5)))).to(torch.bfloat16)
    a = wl.make_activations(shape, 6, DEV)
    ctx = _ctx(H=H, E=E, k=k, I=I, shared_I=shared_I, max_tokens=T, phase=phase, variant=variant, row_gather=row_gather)
    out, bufs = _run_step(ctx, a, w, T)
    ref = _oracle_step(a, w, k)
    emu = _oracle_step(a, w, k, emulate=True)
    N = T * k
    dbg = ctx.moe_ctx_debug_ptrs()
    assert np.array_equal(np_i32(bufs["perm"]), ref["perm"])
    # activation and expert outputs against the oracle's (storage-rounded) stages, valid rows only
    for name, key in (("act", "act"), ("y_perm", "y")):
        e = layer_errors(dbg[name][:N], emu[key])
        scale = np.abs(emu[key]).max()
        assert e["rel_l2"] <= 3e-3 and e["max_abs"] <= 2 ** -7 * scale + 1e-6, f"{vname} {name}: {e}"
    if shared_I:
        e = layer_errors(dbg["y_shared"][:T], emu["y_shared"])
        assert e["rel_l2"] <= 3e-3, f"{vname} y_shared: {e}"
    e = layer_errors(out, ref["out"])
    assert e["rel_l2"] <= 5e-3, f"{vname} out: {e}"
    e2 = layer_errors(out, emu["out"])
    assert e2["rel_l2"] <= 3e-3, f"{vname} out vs storage-rounded oracle: {e2}"
    ctx.close()


def test_combine_alone_matches_oracle():
    """Combine fed with known rows: y_perm written by hand into the workspace, no FFN involved."""
    T, H, E, k = 50, 512, 8, 4
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=64, shared_I=64)
    a = wl.make_activations(shape, 21, DEV)
    w = wl.make_weights(shape, 22, DEV)
    ctx = _ctx(H=H, E=E, k=k, I=64, shared_I=64, max_tokens=T, variant=B.MOE_GEMM_VALIDATION)
    out, bufs = _run_step(ctx, a, w, T)  # defines the layout; then overwrite the rows and combine again
    dbg = ctx.moe_ctx_debug_ptrs()
    g = torch.Generator(device=DEV).manual_seed(23)
    y = torch.randn(T * k, H, generator=g, device=DEV).to(torch.bfloat16)
    ys = torch.randn(T, H, generator=g, device=DEV).to(torch.bfloat16)
    torch.cuda.synchronize()
    ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    dbg["y_perm"][:T * k].copy_(y)
    dbg["y_shared"][:T].copy_(ys)
    torch.cuda.synchronize()
    ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)
    torch.cuda.synchronize()
    ref = oracle.combine(np_f32(y), np_i32(bufs["inv_perm"]), np_f32(bufs["topk_w"]), np_f32(ys))
    got = np_f32(out)
    rounded = oracle.bf16_to_f32(oracle.f32_to_bf16(ref))
    # the only difference allowed is one bf16 rounding of an fp32 sum
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2 ** -8 + 1e-6)
    assert (got != rounded).mean() < 1e-2
    ctx.close()


@pytest.mark.parametrize("phase", [B.MOE_PHASE_DECODE, B.MOE_PHASE_PREFILL])
@pytest.mark.parametrize("T,H,E,k,I,shared_I", [
    (300, 512, 16, 4, 192, 128),   # ragged tiles and a shared expert
    (1100, 256, 3, 2, 128, 0),     # several token chunks per expert
    (90, 320, 40, 8, 64, 0),       # many small experts, some empty
])
def test_the_result_does_not_depend_on_the_number_of_ctas(phase, T, H, E, k, I, shared_I):
    """The small-M kernel deals the first waves of its tile list statically and hands the rest out through an atomic
    counter; whatever the grid -- one CTA, a few, all -- every tile is computed exactly once and the layer's bits
    are the same."""
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    w, a = wl.make_weights(shape, 21, DEV), wl.make_activations(shape, 22, DEV)
    outs = {}
    for budget in (0, 1, 2, 5, 37):
        ctx = _ctx(H=H, E=E, k=k, I=I, shared_I=shared_I, max_tokens=T, phase=phase, variant=B.MOE_GEMM_SMALL_M,
                   sm_budget=budget)
        for rep in range(2):  # twice: the second step finds the counters the first one left
            out, _ = ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
        torch.cuda.synchronize()
        assert ctx.moe_ctx_status() == B.MOE_OK
        outs[budget] = out.clone()
        ctx.close()
    for budget, out in outs.items():
        assert torch.equal(out, outs[0]), f"sm_budget = {budget} changes the result"
