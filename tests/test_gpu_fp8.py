"""FP8 (E4M3) precision variant against the oracle's statement of the same recipe.

Stage by stage, so that every comparison is as tight as its arithmetic allows:
  * the quantisation of the GEMM1 input rows (done per token, then moved) is integer work decided in fp32: codes
    and scales of the permuted rows bit-exact;
  * GEMM1 + SwiGLU from identical codes: the bf16 activation within bf16 rounding of the oracle's;
  * the activation's quantisation, applied by the oracle to the GPU's own activation: bit-exact again;
  * GEMM2 from the GPU's own codes: within bf16 rounding of the oracle's fp64 sums;
  * the whole layer end to end: within the error that one bf16 ulp of difference in the activation can cause
    through its re-quantisation (derived below), and within E4M3's own error of the bf16 layer.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import np_f32, np_i32
from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _np_u8(t):
    return t.detach().cpu().numpy()


def _w8_host(w8):
    return {k: (None if v is None else (_np_u8(v) if v.dtype == torch.uint8 else np_f32(v))) for k, v in w8.items()}


CASES = [
    # T, H, E, k, I, shared_I, phase, variant
    (64, 256, 8, 2, 512, 0, B.MOE_PHASE_PREFILL, B.MOE_GEMM_AUTO),      # the smallest config's shape
    (300, 512, 6, 3, 192, 128, B.MOE_PHASE_PREFILL, B.MOE_GEMM_AUTO),   # ragged tiles, shared expert, K not a multiple of 128
    (48, 512, 16, 4, 256, 128, B.MOE_PHASE_DECODE, B.MOE_GEMM_AUTO),    # decode variant with a shared expert
    (130, 1024, 5, 2, 320, 0, B.MOE_PHASE_PREFILL, B.MOE_GEMM_SMALL_M), # small-M kernel on more rows than one tile
]


@pytest.mark.parametrize("T,H,E,k,I,shared_I,phase,variant", CASES)
def test_fp8_stages_against_the_oracle(T, H, E, k, I, shared_I, phase, variant):
    shape = wl.LayerShape("f8", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=True)
    # weights ~ N(0, 1/sqrt(fan_in)): unit-variance pre-activations, so that an error anywhere is visible
    w8 = wl.make_weights_fp8(shape, 11, DEV, std=1.0)
    for name, fan in (("sw_gate_up", H), ("sws_gate_up", H), ("sw_down", I), ("sws_down", shared_I)):
        if w8[name] is not None:
            w8[name] = (w8[name] / fan ** 0.5).contiguous()
    a = wl.make_activations(shape, 12, DEV)
    ctx = B.MoeContext(B.make_config(H, E, k, I, shared_I, T, phase, 0, variant, weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    torch.cuda.synchronize()
    out, bufs = ctx.layer_fp8(a["x"], a["logits"], a["bias"], w8)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    N = T * k
    dbg = ctx.moe_ctx_debug_ptrs()
    x_perm = oracle.permute(wl.bits(a["x"]), np_i32(bufs["perm"]).reshape(-1), k)  # an FP8 context keeps no bf16 copy
    act_gpu = wl.bits(dbg["act"][:N])
    y_gpu = np_f32(dbg["y_perm"][:N])
    xq_gpu, sx_gpu = _np_u8(ctx.fp8_debug_view("xq", (N, H), torch.uint8)), np_f32(ctx.fp8_debug_view("sx", (N,), torch.float32))
    aq_gpu, sa_gpu = _np_u8(ctx.fp8_debug_view("aq", (N, I), torch.uint8)), np_f32(ctx.fp8_debug_view("sa", (N,), torch.float32))
    h = _w8_host(w8)
    offsets = np_i32(bufs["offsets"])

    # 1. quantisation of the permuted rows: bit-exact
    xq_ref, sx_ref = oracle.quantize_rows(x_perm)
    assert np.array_equal(xq_gpu, xq_ref) and np.array_equal(sx_gpu, sx_ref)

    # 2. GEMM1 + SwiGLU from identical codes, 3. re-quantisation of the GPU's activation, 4. GEMM2 from it
    aq_ref, sa_ref = oracle.quantize_rows(act_gpu)
    assert np.array_equal(aq_gpu, aq_ref) and np.array_equal(sa_gpu, sa_ref)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 == r0:
            continue
        act_ref = oracle.bf16_to_f32(oracle.gemm1_fp8(xq_ref[r0:r1], sx_ref[r0:r1], h["wq_gate_up"][e], h["sw_gate_up"][e]))
        ag = oracle.bf16_to_f32(act_gpu[r0:r1])
        # one bf16 ulp (2^-8 relative) of slack for the fp32 accumulation order and the fast exponential, plus
        # an absolute term for values whose g and u partly cancelled
        assert np.all(np.abs(ag - act_ref) <= 2.0 ** -7 * np.abs(act_ref) + 2e-3), f"GEMM1 expert {e}"
        y_ref = oracle.gemm2_fp8(aq_gpu[r0:r1], sa_gpu[r0:r1], h["wq_down"][e], h["sw_down"][e])
        assert np.all(np.abs(y_gpu[r0:r1] - y_ref) <= 2.0 ** -8 * np.abs(y_ref) + 2e-3), f"GEMM2 expert {e}"

    # 5. end to end.  The GPU's activation differs from the oracle's by at most a bf16 ulp (2^-8) on a few
    # elements; where that moves an element across an E4M3 rounding boundary its code changes by one step
    # (2^-3 relative at worst), which happens to a fraction ~2^-8 / 2^-4 = 6 % of the differing elements.  With
    # at most every element differing, the relative L2 error of y is bounded by sqrt(0.06) * 2^-4 / sqrt(3)
    # ~ 0.9 % in the worst case.  Measured: 0.23 %, which is the bf16 rounding of the output itself, so the
    # layer's own tolerance (relative L2 <= 5e-3) is asserted here too.
    ref = oracle.layer_fp8(wl.bits(a["x"]), np_f32(a["logits"]), np_f32(a["bias"]), k, h["wq_gate_up"], h["sw_gate_up"],
                           h["wq_down"], h["sw_down"], h["wsq_gate_up"], h["sws_gate_up"], h["wsq_down"], h["sws_down"])
    for name in ("topk_idx", "counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(np_i32(bufs[name]).reshape(-1), np.asarray(ref[name]).reshape(-1)), name
    rel = np.linalg.norm(np_f32(out) - ref["out"]) / np.linalg.norm(ref["out"])
    print(f"[fp8 parity T={T} H={H} E={E}] rel_l2={rel:.4g}")
    assert rel <= 5e-3, rel
    ctx.close()


def test_fp8_call_is_refused_on_a_bf16_context_and_the_other_way_round():
    shape = wl.LayerShape("f8", T=32, H=256, E=8, k=2, I=128)
    w8, w16, a = wl.make_weights_fp8(shape, 1, DEV), wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(256, 8, 2, 128, 0, 32))
    with pytest.raises(B.MoeError) as ei:
        ctx.layer_fp8(a["x"], a["logits"], None, w8)
    assert ei.value.status == B.MOE_ERR_STATE
    ctx.moe_ctx_abandon_step()
    out, _ = ctx.layer(a["x"], a["logits"], None, w16["w_gate_up"], w16["w_down"])  # still usable
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.close()
    with pytest.raises(B.MoeError):  # the CUDA-core check kernel has no FP8 form
        B.MoeContext(B.make_config(256, 8, 2, 128, 0, 32, gemm_variant=B.MOE_GEMM_VALIDATION,
                                   weight_format=B.MOE_WEIGHTS_FP8_E4M3))


def test_fp8_decode_step_replays_from_a_cuda_graph_and_is_run_to_run_identical():
    shape = wl.LayerShape("f8", T=48, H=512, E=16, k=4, I=256, shared_I=128, select_bias=True)
    w8 = wl.make_weights_fp8(shape, 1, DEV)
    a1, a2 = wl.make_activations(shape, 2, DEV), wl.make_activations(shape, 3, DEV)
    sd = torch.cuda.Stream()
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 48, B.MOE_PHASE_DECODE,
                                   weight_format=B.MOE_WEIGHTS_FP8_E4M3), stream=sd)
    torch.cuda.synchronize()
    eager1, _ = d.layer_fp8(a1["x"], a1["logits"], a1["bias"], w8)
    eager2, _ = d.layer_fp8(a2["x"], a2["logits"], a2["bias"], w8)
    again1, _ = d.layer_fp8(a1["x"], a1["logits"], a1["bias"], w8)   # the other buffer set, same bits
    torch.cuda.synchronize()
    assert torch.equal(again1, eager1)
    x, logits, bias = a1["x"].clone(), a1["logits"].clone(), a1["bias"].clone()
    bufs = B.alloc_step_buffers(48, 4, 16, DEV)
    out = torch.empty(48, 512, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=sd):
        d.layer_fp8(x, logits, bias, w8, out=out, bufs=bufs)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager1)
    x.copy_(a2["x"]); logits.copy_(a2["logits"]); bias.copy_(a2["bias"])
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager2)
    assert d.moe_ctx_status() == B.MOE_OK
    del g
    d.close()


_V3_FP8 = {}


def _v3_fp8_weights():
    """One copy of the V3-shaped FP8 weights (11.4 GB) for both phases' tests."""
    if not _V3_FP8:
        shape = wl.C4_D
        w8 = wl.make_weights_fp8(shape, 21, DEV, std=1.0)
        for name, fan in (("sw_gate_up", shape.H), ("sws_gate_up", shape.H), ("sw_down", shape.I),
                          ("sws_down", shape.shared_I)):
            w8[name] = (w8[name] / fan ** 0.5).contiguous()
        _V3_FP8.update(w8)
    return _V3_FP8


@pytest.mark.parametrize("shape,phase", [(wl.C4_D, B.MOE_PHASE_DECODE), (wl.C4_P, B.MOE_PHASE_PREFILL)],
                         ids=["decode-T64", "prefill-T4096"])
def test_fp8_at_the_v3_layer_shape_on_sampled_tokens(shape, phase):
    """Both batches of config 4 on the DeepSeek-V3-shaped layer (H=7168, E=256, top-8, I=2048, shared expert) with
    FP8 weights: 56 k-blocks per GEMM1 tile, the small-M kernel for D and the large-M kernel for P, the shared
    expert riding along.  The oracle follows sampled tokens through their eight experts (only those experts'
    codes leave the GPU)."""
    T, H, E, k, I, Is = shape.T, shape.H, shape.E, shape.k, shape.I, shape.shared_I
    w8 = _v3_fp8_weights()
    a = wl.make_activations(shape, 22, DEV)
    ctx = B.MoeContext(B.make_config(H, E, k, I, Is, T, phase, weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    torch.cuda.synchronize()
    out, bufs = ctx.layer_fp8(a["x"], a["logits"], a["bias"], w8)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    idx_ref, w_ref = oracle.route(np_f32(a["logits"]), np_f32(a["bias"]), k)
    assert np.array_equal(np_i32(bufs["topk_idx"]), idx_ref)
    x_bits = wl.bits(a["x"])
    shared = [_np_u8(w8["wsq_gate_up"]), np_f32(w8["sws_gate_up"]), _np_u8(w8["wsq_down"]), np_f32(w8["sws_down"])]
    out_gpu = np_f32(out)
    for t in (0, (17 * T) // 64, T - 1):
        acc = oracle.ffn_fp8(x_bits[t:t + 1], *shared)[0].astype(np.float64)
        for j in range(k):
            e = int(idx_ref[t, j])
            y = oracle.ffn_fp8(x_bits[t:t + 1], _np_u8(w8["wq_gate_up"][e]), np_f32(w8["sw_gate_up"][e]),
                               _np_u8(w8["wq_down"][e]), np_f32(w8["sw_down"][e]))[0]
            acc += float(w_ref[t, j]) * y.astype(np.float64)
        rel = np.linalg.norm(out_gpu[t] - acc) / np.linalg.norm(acc)
        print(f"[fp8 parity V3 shape T={T}, token {t}] rel_l2={rel:.4g}")
        assert rel <= 5e-3, (t, rel)
    ctx.close()


def test_fp8_prefill_segments_are_bit_identical_and_boundaries_are_counted():
    shape = wl.LayerShape("f8", T=300, H=512, E=6, k=3, I=192, shared_I=128, select_bias=True)
    w8, a = wl.make_weights_fp8(shape, 5, DEV), wl.make_activations(shape, 6, DEV)
    ctx = B.MoeContext(B.make_config(512, 6, 3, 192, 128, 300, B.MOE_PHASE_PREFILL,
                                     weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    torch.cuda.synchronize()
    whole, _ = ctx.layer_fp8(a["x"], a["logits"], a["bias"], w8)
    whole = whole.clone()
    seen = []
    ctx.moe_ctx_set_segments(2, lambda i, n: seen.append((i, n)))
    cut, _ = ctx.layer_fp8(a["x"], a["logits"], a["bias"], w8)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    assert torch.equal(cut, whole)
    # 3 routed segments per pass, the shared expert's two passes and the activation's quantisation
    assert seen == [(i, 9) for i in range(9)]
    ctx.close()


def test_entry_points_that_do_not_serve_an_fp8_context_say_so():
    shape = wl.LayerShape("f8", T=16, H=256, E=4, k=2, I=128)
    w16, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(256, 4, 2, 128, 0, 16, weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    hx, hl = a["x"].cpu().pin_memory(), a["logits"].cpu().pin_memory()
    hout = torch.empty(16, 256, dtype=torch.bfloat16).pin_memory()
    for call in (lambda: ctx.moe_layer_host_submit(0, hl, None, hx, w16["w_gate_up"], w16["w_down"], None, None, hout),
                 lambda: ctx.moe_layer_host(hl, None, hx, w16["w_gate_up"], w16["w_down"], None, None, hout)):
        with pytest.raises(B.MoeError) as ei:
            call()
        assert ei.value.status == B.MOE_ERR_STATE
    # the context is between steps after either refusal and still runs an FP8 step
    w8 = wl.make_weights_fp8(shape, 3, DEV)
    out, _ = ctx.layer_fp8(a["x"], a["logits"], None, w8)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK and torch.isfinite(out.float()).all()
    with pytest.raises(B.MoeError):  # the row gather has no FP8 form
        B.MoeContext(B.make_config(256, 4, 2, 128, 0, 16, row_gather=1, weight_format=B.MOE_WEIGHTS_FP8_E4M3))
    ctx.close()
