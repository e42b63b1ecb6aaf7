"""Phase contexts: ownership, isolation, call order and host-side error paths (no GPU is ever faulted)."""
import ctypes
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import check_layer, layer_errors, np_f32, np_i32
from paper_2609_00993_b200 import binding as B
from paper_2609_00993_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _cfg(phase=B.MOE_PHASE_PREFILL, max_tokens=32, **kw):
    return B.make_config(256, 8, 2, 128, kw.pop("shared_inter", 0), max_tokens, phase, **kw)


def test_workspaces_of_live_contexts_may_not_overlap():
    cfg = _cfg()
    n = B.moe_ctx_workspace_bytes(cfg)
    ws = torch.empty(2 * n + 512, dtype=torch.uint8, device=DEV)
    a = B.MoeContext(cfg, workspace=ws[:n])
    with pytest.raises(B.MoeError) as ei:
        B.MoeContext(cfg, workspace=ws[256:256 + n])
    assert ei.value.status == B.MOE_ERR_STATE
    off = (n + 255) // 256 * 256
    b = B.MoeContext(cfg, workspace=ws[off:off + n])  # disjoint range: fine
    a.close(); b.close()
    c = B.MoeContext(cfg, workspace=ws[256:256 + n])  # the range is free again after destroy
    c.close()


def test_a_stream_serves_one_phase_only():
    s = torch.cuda.Stream()
    p = B.MoeContext(_cfg(B.MOE_PHASE_PREFILL), stream=s)
    with pytest.raises(B.MoeError) as ei:
        B.MoeContext(_cfg(B.MOE_PHASE_DECODE), stream=s)
    assert ei.value.status == B.MOE_ERR_STATE
    p.close()


def test_decode_context_holds_two_buffer_sets():
    staging = 32 * 8 * 4 + 2 * 32 * 256 * 2  # one extra host-staging slot (P carves three, D two)
    assert (B.moe_ctx_workspace_bytes(_cfg(B.MOE_PHASE_DECODE)) - 2 * staging
            > 1.9 * (B.moe_ctx_workspace_bytes(_cfg()) - 3 * staging) - 4096)
    ctx = B.MoeContext(_cfg(B.MOE_PHASE_DECODE))
    shape = wl.LayerShape("t", T=32, H=256, E=8, k=2, I=128)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    torch.cuda.synchronize()
    ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    p1 = ctx.moe_ctx_debug_ptrs()["y_perm"].data_ptr()
    ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    p2 = ctx.moe_ctx_debug_ptrs()["y_perm"].data_ptr()
    ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    p3 = ctx.moe_ctx_debug_ptrs()["y_perm"].data_ptr()
    assert p1 != p2 and p1 == p3  # the double-buffer index flips per step; addresses are stable
    ctx.close()


def test_call_order_and_argument_errors():
    ctx = B.MoeContext(_cfg())
    shape = wl.LayerShape("t", T=32, H=256, E=8, k=2, I=128)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    bufs = B.alloc_step_buffers(32, 2, 8, DEV)
    out = torch.empty(32, 256, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()

    def status_of(fn):
        with pytest.raises(B.MoeError) as ei:
            fn()
        return ei.value.status

    assert status_of(lambda: ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)) == B.MOE_ERR_STATE
    assert status_of(lambda: ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"])) == B.MOE_ERR_STATE
    big = torch.zeros(64, 8, device=DEV)
    assert status_of(lambda: ctx.moe_route(big, None, bufs["topk_idx"], bufs["topk_w"])) == B.MOE_ERR_CAPACITY
    odd = torch.zeros(32 * 8 + 4, device=DEV)[1:257].view(32, 8)  # 4 bytes past a 16-byte boundary
    assert status_of(lambda: ctx.moe_route(odd, None, bufs["topk_idx"], bufs["topk_w"])) == B.MOE_ERR_INVALID_ARG
    ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])
    ctx.moe_dispatch_layout(bufs["topk_idx"], None)  # layout only
    assert status_of(lambda: ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"])) == B.MOE_ERR_STATE
    ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"])
    assert status_of(lambda: ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])) == B.MOE_ERR_STATE
    assert status_of(lambda: ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], T=16)) == B.MOE_ERR_INVALID_ARG
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"])
    ctx.moe_combine(bufs["topk_w"], None, out)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    assert ctx.moe_ctx_launch_count() >= 5
    ctx.close()


def test_an_abandoned_step_leaves_the_context_usable_and_rests_its_buffer_set():
    """Lifetime rule of Section "Network and Lifetime Isolation": an abandoned operation retires its buffer."""
    shape = wl.LayerShape("t", T=32, H=256, E=8, k=2, I=128)
    w = wl.make_weights(shape, 1, DEV)
    a, a2 = wl.make_activations(shape, 2, DEV), wl.make_activations(shape, 3, DEV)
    torch.cuda.synchronize()
    for phase in (B.MOE_PHASE_PREFILL, B.MOE_PHASE_DECODE):
        ctx = B.MoeContext(_cfg(phase))
        bufs = B.alloc_step_buffers(32, 2, 8, DEV)
        ctx.moe_ctx_abandon_step()  # nothing in progress: a no-op
        ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])
        ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"])
        abandoned = ctx.moe_ctx_debug_ptrs()["x_perm"].data_ptr()
        with pytest.raises(B.MoeError):  # mid-step: a new step may not begin ...
            ctx.moe_route(a2["logits"], None, bufs["topk_idx"], bufs["topk_w"])
        ctx.moe_ctx_abandon_step()       # ... until the step is given up
        out, _ = ctx.layer(a2["x"], a2["logits"], None, w["w_gate_up"], w["w_down"])
        used = ctx.moe_ctx_debug_ptrs()["x_perm"].data_ptr()
        torch.cuda.synchronize()
        assert ctx.moe_ctx_status() == B.MOE_OK
        if phase == B.MOE_PHASE_DECODE:
            assert used != abandoned  # the next step worked in the other buffer set
        ref = oracle.layer(wl.bits(a2["x"]), np_f32(a2["logits"]), None, 2, wl.bits(w["w_gate_up"]),
                           wl.bits(w["w_down"]))
        check_layer(out, ref["out"], label="after an abandoned step")
        ctx.close()


def test_pipelined_host_path_overlaps_steps_and_matches_the_device_path():
    """moe_layer_host_submit / moe_layer_host_wait: results equal the device path's bit for bit, in submission
    order, on both phases; a slot cannot be resubmitted before it was waited for."""
    shape = wl.LayerShape("t", T=32, H=256, E=8, k=2, I=128, shared_I=64, select_bias=True)
    w = wl.make_weights(shape, 1, DEV)
    acts = [wl.make_activations(shape, 10 + i, DEV) for i in range(5)]
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    for phase in (B.MOE_PHASE_PREFILL, B.MOE_PHASE_DECODE):
        ctx = B.MoeContext(_cfg(phase, shared_inter=64), stream=torch.cuda.Stream())
        ref = []
        for a in acts:
            o, _ = ctx.layer(a["x"], a["logits"], a["bias"], *wargs)
            ref.append(o.clone())
        torch.cuda.synchronize()
        hx = [a["x"].cpu().pin_memory() for a in acts]
        hl = [a["logits"].cpu().pin_memory() for a in acts]
        hout = [torch.zeros(32, 256, dtype=torch.bfloat16).pin_memory() for _ in acts]
        n_slots = 3  # any number up to MOE_HOST_SLOTS = 4
        for i in range(n_slots):
            ctx.moe_layer_host_submit(i, hl[i], acts[i]["bias"], hx[i], *wargs, hout[i])
        with pytest.raises(B.MoeError) as ei:  # slot 1 has not been waited for
            ctx.moe_layer_host_submit(1, hl[3], acts[3]["bias"], hx[3], *wargs, hout[3])
        assert ei.value.status == B.MOE_ERR_STATE
        with pytest.raises(B.MoeError) as ei:
            ctx.moe_layer_host_submit(4, hl[3], acts[3]["bias"], hx[3], *wargs, hout[3])
        assert ei.value.status == B.MOE_ERR_INVALID_ARG
        for i in range(n_slots, 5):
            ctx.moe_layer_host_wait(i % n_slots)
            assert torch.equal(hout[i - n_slots], ref[i - n_slots].cpu())
            ctx.moe_layer_host_submit(i % n_slots, hl[i], acts[i]["bias"], hx[i], *wargs, hout[i])
        for sl in range(4):
            ctx.moe_layer_host_wait(sl)  # slot 3 never had anything in flight: a no-op
        for i in range(5):
            assert torch.equal(hout[i], ref[i].cpu())
        assert ctx.moe_ctx_status() == B.MOE_OK
        ctx.close()


def test_create_rejects_bad_configurations():
    for bad in (B.make_config(100, 8, 2, 128, 0, 4), B.make_config(256, 8, 9, 128, 0, 4),
                B.make_config(256, 2000, 2, 128, 0, 4), B.make_config(256, 8, 2, 128, 0, 0)):
        assert B.moe_ctx_workspace_bytes(bad) == 0
        with pytest.raises(B.MoeError):
            B.MoeContext(bad)
    cfg = _cfg()
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    lib = B.load_library()
    h = ctypes.c_void_p()
    st = lib.moe_ctx_create(ctypes.byref(cfg), ctypes.c_void_p(small.data_ptr()), small.numel(), None, ctypes.byref(h))
    assert st == B.MOE_ERR_CAPACITY and not h.value


def test_destroy_refuses_while_work_is_in_flight():
    """An abandoned operation retires its buffers only at a quiescent point."""
    shape = wl.C3.with_tokens(4096)
    cfg = B.make_config(shape.H, shape.E, shape.k, shape.I, 0, shape.T, B.MOE_PHASE_PREFILL, 0, B.MOE_GEMM_VALIDATION)
    s = torch.cuda.Stream()
    ctx = B.MoeContext(cfg, stream=s)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    torch.cuda.synchronize()
    for _ in range(3):
        ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])  # the slow validation GEMM keeps the stream busy
    with pytest.raises(B.MoeError) as ei:
        ctx.destroy()
    assert ei.value.status == B.MOE_ERR_STATE
    s.synchronize()
    ctx.destroy()


def test_prefill_traffic_cannot_disturb_a_decode_step():
    """P runs between D's layout and D's combine; D's results are bit-identical to D alone."""
    shape = wl.LayerShape("t", T=64, H=512, E=16, k=4, I=256, shared_I=128)
    pshape = shape.with_tokens(1024)
    w = wl.make_weights(shape, 1, DEV)
    ad, ap = wl.make_activations(shape, 2, DEV), wl.make_activations(pshape, 3, DEV)
    sp, sd = torch.cuda.Stream(), torch.cuda.Stream()
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 64, B.MOE_PHASE_DECODE), stream=sd)
    p = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 1024, B.MOE_PHASE_PREFILL), stream=sp)
    torch.cuda.synchronize()
    alone, bufs_alone = d.layer(ad["x"], ad["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    d.layer(ad["x"], ad["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])  # back to buffer set 0
    torch.cuda.synchronize()
    bufs = B.alloc_step_buffers(64, 4, 16, DEV)
    out = torch.empty(64, 512, dtype=torch.bfloat16, device=DEV)
    d.moe_route(ad["logits"], None, bufs["topk_idx"], bufs["topk_w"])
    d.moe_dispatch_layout(bufs["topk_idx"], ad["x"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    for _ in range(3):
        p.layer(ap["x"], ap["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    d.moe_grouped_ffn(w["w_gate_up"], w["w_down"], ad["x"], w["ws_gate_up"], w["ws_down"])
    p.layer(ap["x"], ap["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    d.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)
    torch.cuda.synchronize()
    assert torch.equal(out, alone)
    assert torch.equal(bufs["perm"], bufs_alone["perm"])
    p.close(); d.close()


def test_prefill_segments_are_bit_identical_and_boundaries_are_monotone():
    shape = wl.LayerShape("t", T=600, H=512, E=16, k=4, I=256, shared_I=128)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 600, B.MOE_PHASE_PREFILL))
    torch.cuda.synchronize()
    whole, _ = ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    for span in (1, 5, 16, 64):
        seen = []
        ctx.moe_ctx_set_segments(span, lambda i, n: seen.append((i, n)))
        out, _ = ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
        torch.cuda.synchronize()
        assert torch.equal(out, whole), f"span {span}"
        segs = -(-16 // min(span, 16))
        assert seen == [(i, 2 * segs + 2) for i in range(2 * segs + 2)], f"span {span}: {seen}"
    ctx.moe_ctx_set_segments(0)
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.close()


def test_decode_step_admitted_at_a_prefill_boundary():
    """The host controller enqueues a D step at a P boundary and holds P's next segment until D is done:
    both phases give exactly the results they give alone."""
    shape = wl.LayerShape("t", T=48, H=512, E=16, k=4, I=256, shared_I=128)
    pshape = shape.with_tokens(2048)
    w = wl.make_weights(shape, 1, DEV)
    ad, ap = wl.make_activations(shape, 2, DEV), wl.make_activations(pshape, 3, DEV)
    sp, sd = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 48, B.MOE_PHASE_DECODE), stream=sd)
    p = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 2048, B.MOE_PHASE_PREFILL), stream=sp)
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    d_alone, _ = d.layer(ad["x"], ad["logits"], None, *wargs)
    p_alone, _ = p.layer(ap["x"], ap["logits"], None, *wargs)
    torch.cuda.synchronize()
    d_out = torch.empty_like(d_alone)
    admitted = []

    def turnstile(i, n):
        if i % 3 == 0:  # admit one D step at every third boundary
            d.layer(ad["x"], ad["logits"], None, *wargs, out=d_out)
            ev = torch.cuda.Event()
            ev.record(sd)
            sp.wait_event(ev)  # the next P segment starts after this D step
            admitted.append(i)

    p.moe_ctx_set_segments(4, turnstile)
    p_out, _ = p.layer(ap["x"], ap["logits"], None, *wargs)
    torch.cuda.synchronize()
    assert len(admitted) == 4 and admitted[0] == 0  # 2 * 4 + 2 = 10 boundaries
    assert torch.equal(p_out, p_alone) and torch.equal(d_out, d_alone)
    assert p.moe_ctx_status() == B.MOE_OK and d.moe_ctx_status() == B.MOE_OK
    p.moe_ctx_set_segments(0)
    p.close(); d.close()


def test_split_dispatch_state_transitions():
    """Notification and row movement as two calls: at most one pending dispatch per context, explicit transitions,
    an abandoned step retires the pending dispatch, and the one-call and two-call forms give the same bits."""
    shape = wl.LayerShape("t", T=300, H=256, E=8, k=2, I=128, shared_I=64)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(256, 8, 2, 128, 64, 300, B.MOE_PHASE_PREFILL))
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    whole, wb = ctx.layer(a["x"], a["logits"], None, *wargs)
    torch.cuda.synchronize()
    bufs = B.alloc_step_buffers(300, 2, 8, DEV)
    out = torch.empty_like(whole)
    assert ctx.moe_ctx_pending_dispatch() == {"pending": False, "tokens": 0, "notified_done": False}
    with pytest.raises(B.MoeError) as ei:      # no pending dispatch to move
        ctx.moe_dispatch_move(a["x"])
    assert ei.value.status == B.MOE_ERR_STATE
    ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])
    ctx.moe_dispatch_notify(bufs["topk_idx"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_pending_dispatch() == {"pending": True, "tokens": 300, "notified_done": True}
    # the integer results are complete after the first half
    ref = oracle.layout(np_i32(bufs["topk_idx"]).reshape(-1), 8)
    for name, want in zip(("counts", "offsets", "perm", "inv_perm"), ref):
        assert np.array_equal(np_i32(bufs[name]), want), name
    for call in (lambda: ctx.moe_dispatch_notify(bufs["topk_idx"]),                 # a second notification
                 lambda: ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"]),         # the one-call form
                 lambda: ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"]),
                 lambda: ctx.moe_route(a["logits"], None, bufs["topk_idx"], bufs["topk_w"])):
        with pytest.raises(B.MoeError) as ei:
            call()
        assert ei.value.status == B.MOE_ERR_STATE
    assert ctx.moe_ctx_pending_dispatch()["pending"]
    ctx.moe_dispatch_move(a["x"])
    assert not ctx.moe_ctx_pending_dispatch()["pending"]
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"])
    ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)
    torch.cuda.synchronize()
    assert torch.equal(out, whole) and torch.equal(bufs["perm"], wb["perm"])
    # abandoning a step retires its pending dispatch; the context then takes a new notification
    ctx.moe_dispatch_notify(bufs["topk_idx"])
    ctx.moe_ctx_abandon_step()
    assert not ctx.moe_ctx_pending_dispatch()["pending"]
    ctx.moe_dispatch_notify(bufs["topk_idx"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    ctx.moe_dispatch_move(a["x"])
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"])
    ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)
    torch.cuda.synchronize()
    assert torch.equal(out, whole) and ctx.moe_ctx_status() == B.MOE_OK
    # with segmentation on, the notification is boundary 0 and the FFN's boundaries follow it
    seen = []
    ctx.moe_ctx_set_segments(4, lambda i, n: seen.append((i, n)))
    ctx.moe_dispatch_notify(bufs["topk_idx"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
    assert seen == [(0, 7)]                       # 1 + 2 * 2 routed segments + 2 shared-expert passes
    ctx.moe_dispatch_move(a["x"])
    ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"])
    ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)
    torch.cuda.synchronize()
    assert seen == [(i, 7) for i in range(7)] and torch.equal(out, whole)
    ctx.moe_ctx_set_segments(0)
    ctx.close()


@pytest.mark.parametrize("fmt", [B.MOE_WEIGHTS_BF16, B.MOE_WEIGHTS_FP8_E4M3])
def test_decode_step_admitted_between_notification_and_row_movement(fmt):
    """The first safe point of a prefill step: P has enqueued its layout (notification, counts, permutation) and
    holds a pending dispatch; the controller admits a whole D step there and gives P's row movement its permit
    only afterwards.  Both phases give the bits they give alone, and those match the oracle."""
    shape = wl.LayerShape("t", T=40, H=512, E=16, k=4, I=256, shared_I=128, select_bias=True)
    pshape = shape.with_tokens(1500)
    fp8 = fmt == B.MOE_WEIGHTS_FP8_E4M3
    w = wl.make_weights_fp8(shape, 1, DEV) if fp8 else wl.make_weights(shape, 1, DEV)
    ad, ap = wl.make_activations(shape, 2, DEV), wl.make_activations(pshape, 3, DEV)
    sp, sd = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 40, B.MOE_PHASE_DECODE, weight_format=fmt), stream=sd)
    p = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 1500, B.MOE_PHASE_PREFILL, weight_format=fmt), stream=sp)

    def ffn(ctx, a, T):
        if fp8:
            ctx.moe_grouped_ffn_fp8(w["wq_gate_up"], w["sw_gate_up"], w["wq_down"], w["sw_down"], w["wsq_gate_up"],
                                    w["sws_gate_up"], w["wsq_down"], w["sws_down"], T=T)
        else:
            ctx.moe_grouped_ffn(w["w_gate_up"], w["w_down"], a["x"], w["ws_gate_up"], w["ws_down"])

    def whole_step(ctx, a, out, bufs):
        T = a["x"].shape[0]
        ctx.moe_route(a["logits"], a["bias"], bufs["topk_idx"], bufs["topk_w"])
        ctx.moe_dispatch_layout(bufs["topk_idx"], a["x"], bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"])
        ffn(ctx, a, T)
        ctx.moe_combine(bufs["topk_w"], bufs["inv_perm"], out)

    bd, bp = B.alloc_step_buffers(40, 4, 16, DEV), B.alloc_step_buffers(1500, 4, 16, DEV)
    d_alone, p_alone = torch.empty(40, 512, dtype=torch.bfloat16, device=DEV), torch.empty(1500, 512, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    with torch.cuda.stream(sd):
        whole_step(d, ad, d_alone, bd)
    with torch.cuda.stream(sp):
        whole_step(p, ap, p_alone, bp)
    torch.cuda.synchronize()
    d_out, p_out = torch.zeros_like(d_alone), torch.zeros_like(p_alone)
    torch.cuda.synchronize()
    # P: route + notification; then the D step is admitted; then P's rows move behind it
    p.moe_route(ap["logits"], ap["bias"], bp["topk_idx"], bp["topk_w"])
    p.moe_dispatch_notify(bp["topk_idx"], bp["counts"], bp["offsets"], bp["perm"], bp["inv_perm"])
    assert p.moe_ctx_pending_dispatch()["pending"]
    with torch.cuda.stream(sd):
        whole_step(d, ad, d_out, bd)
        ev = torch.cuda.Event()
        ev.record(sd)
    sp.wait_event(ev)                 # the permit: P's data movement is ordered after the D step
    p.moe_dispatch_move(ap["x"])
    ffn(p, ap, 1500)
    p.moe_combine(bp["topk_w"], bp["inv_perm"], p_out)
    torch.cuda.synchronize()
    assert p.moe_ctx_status() == B.MOE_OK and d.moe_ctx_status() == B.MOE_OK
    assert torch.equal(p_out, p_alone) and torch.equal(d_out, d_alone)
    if not fp8:
        for a, out, shp in ((ap, p_out, pshape), (ad, d_out, shape)):
            ref = oracle.layer(wl.bits(a["x"]), np_f32(a["logits"]), np_f32(a["bias"]), 4, wl.bits(w["w_gate_up"]),
                               wl.bits(w["w_down"]), wl.bits(w["ws_gate_up"]), wl.bits(w["ws_down"]))
            e = layer_errors(out, ref["out"])
            assert e["rel_l2"] <= 5e-3 and e["max_abs"] <= 2e-2, e
    p.close(); d.close()


@pytest.mark.parametrize("fmt", [B.MOE_WEIGHTS_BF16, B.MOE_WEIGHTS_FP8_E4M3])
def test_prefill_pass_yields_between_tiles_and_resumes_bit_identically(fmt):
    """Preemption at tile granularity: a second host thread raises yield requests at random moments while P
    steps run; the boundary hook (on P's thread) runs a whole D step on the other stream, lowers the request
    and returns; the pass resumes.  Every P and every D result equals the one computed alone, bit for bit."""
    import random
    import threading
    import time
    fp8 = fmt == B.MOE_WEIGHTS_FP8_E4M3
    shape = wl.LayerShape("t", T=32, H=1024, E=32, k=4, I=512, shared_I=256, select_bias=True)
    pshape = shape.with_tokens(3000)
    w = wl.make_weights_fp8(shape, 1, DEV) if fp8 else wl.make_weights(shape, 1, DEV)
    ad, ap = wl.make_activations(shape, 2, DEV), wl.make_activations(pshape, 3, DEV)
    sp, sd = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    d = B.MoeContext(B.make_config(1024, 32, 4, 512, 256, 32, B.MOE_PHASE_DECODE, weight_format=fmt), stream=sd)
    p = B.MoeContext(B.make_config(1024, 32, 4, 512, 256, 3000, B.MOE_PHASE_PREFILL, weight_format=fmt), stream=sp)
    bd, bp = B.alloc_step_buffers(32, 4, 32, DEV), B.alloc_step_buffers(3000, 4, 32, DEV)
    d_out, p_out = (torch.empty(32, 1024, dtype=torch.bfloat16, device=DEV),
                    torch.empty(3000, 1024, dtype=torch.bfloat16, device=DEV))

    def step(ctx, a, out, bufs):
        if fp8:
            ctx.layer_fp8(a["x"], a["logits"], a["bias"], w, out=out, bufs=bufs)
        else:
            ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"],
                      out=out, bufs=bufs)

    torch.cuda.synchronize()
    with torch.cuda.stream(sd):
        step(d, ad, d_out, bd)
    with torch.cuda.stream(sp):
        step(p, ap, p_out, bp)
    torch.cuda.synchronize()
    d_alone, p_alone = d_out.clone(), p_out.clone()
    assert p.moe_ctx_request_yield(True) == B.MOE_ERR_STATE   # preemption has not been switched on
    p.moe_ctx_set_preemption(True)
    d_runs = []

    def hook(i, n):
        assert i == B.MOE_BOUNDARY_YIELD
        d_out.zero_()
        with torch.cuda.stream(sd):
            step(d, ad, d_out, bd)
        sd.synchronize()
        d_runs.append(torch.equal(d_out, d_alone))
        p.moe_ctx_request_yield(False)     # the permit: P may go on

    p.moe_ctx_set_segments(0, hook)
    rng = random.Random(5)
    stop = threading.Event()

    def requester():
        while not stop.is_set():
            time.sleep(rng.uniform(0.0, 0.0015))
            p.moe_ctx_request_yield(True)
            time.sleep(0.0005)

    th = threading.Thread(target=requester, daemon=True)
    th.start()
    try:
        for it in range(40):
            p_out.zero_()
            with torch.cuda.stream(sp):
                step(p, ap, p_out, bp)
            sp.synchronize()
            assert torch.equal(p_out, p_alone), f"P step {it} differs after {p.moe_ctx_yield_count()} yields"
    finally:
        stop.set()
        th.join()
        p.moe_ctx_request_yield(False)
    assert p.moe_ctx_yield_count() >= 1 and d_runs and all(d_runs)
    assert p.moe_ctx_status() == B.MOE_OK and d.moe_ctx_status() == B.MOE_OK
    # with the request permanently up and a hook that never lowers it, a pass still ends
    p.moe_ctx_set_segments(0, lambda i, n: None)
    p.moe_ctx_request_yield(True)
    p_out.zero_()
    with torch.cuda.stream(sp):
        step(p, ap, p_out, bp)
    sp.synchronize()
    assert torch.equal(p_out, p_alone)
    p.moe_ctx_request_yield(False)
    p.moe_ctx_set_preemption(False)
    p.close(); d.close()
    # the same on four CTAs, where a launch that stops at once gets through four tiles: a request that stays up is
    # honoured 64 times per pass and then overridden by a launch that runs to the pass's end
    p4 = B.MoeContext(B.make_config(1024, 32, 4, 512, 256, 3000, B.MOE_PHASE_PREFILL, sm_budget=4, weight_format=fmt),
                      stream=sp)
    p4.moe_ctx_set_preemption(True)
    p4.moe_ctx_set_segments(0, lambda i, n: None)
    p4.moe_ctx_request_yield(True)
    p_out.zero_()
    with torch.cuda.stream(sp):
        step(p4, ap, p_out, bp)
    sp.synchronize()
    assert p4.moe_ctx_yield_count() >= 128   # 64 in each of the two passes
    assert torch.equal(p_out, p_alone)
    p4.moe_ctx_request_yield(False)
    assert p4.moe_ctx_status() == B.MOE_OK
    p4.close()


@pytest.mark.parametrize("phase,T", [(B.MOE_PHASE_DECODE, 48), (B.MOE_PHASE_PREFILL, 700)])
@pytest.mark.parametrize("fmt", [B.MOE_WEIGHTS_BF16, B.MOE_WEIGHTS_FP8_E4M3])
def test_steps_enqueued_back_to_back_equal_the_same_steps_run_one_at_a_time(phase, T, fmt):
    """Every kernel is launched with the programmatic launch overlap, and the small-M GEMM builds its tile list and
    requests weight boxes before it waits for the previous kernel of the stream.  Steps whose routing differs,
    enqueued right behind one another without a host synchronisation, must give the bits each gives by itself."""
    shape = wl.LayerShape("t", T=T, H=512, E=16, k=4, I=256, shared_I=128, select_bias=True)
    fp8 = fmt == B.MOE_WEIGHTS_FP8_E4M3
    w = wl.make_weights_fp8(shape, 1, DEV) if fp8 else wl.make_weights(shape, 1, DEV)
    acts = [wl.make_activations(shape, 40 + i, DEV) for i in range(4)]  # four different routings
    stream = torch.cuda.Stream()
    ctx = B.MoeContext(B.make_config(512, 16, 4, 256, 128, T, phase, weight_format=fmt), stream=stream)

    def step(a, out, bufs):
        if fp8:
            ctx.layer_fp8(a["x"], a["logits"], a["bias"], w, out=out, bufs=bufs)
        else:
            ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"],
                      out=out, bufs=bufs)

    bufs = [B.alloc_step_buffers(T, 4, 16, DEV) for _ in acts]
    alone = [torch.empty(T, 512, dtype=torch.bfloat16, device=DEV) for _ in acts]
    counts_alone = []
    torch.cuda.synchronize()
    for a, o, b in zip(acts, alone, bufs):
        with torch.cuda.stream(stream):
            step(a, o, b)
        torch.cuda.synchronize()
        counts_alone.append(b["counts"].clone())
    assert not torch.equal(counts_alone[0], counts_alone[1])  # the routing really changes from step to step
    outs = [torch.zeros_like(o) for o in alone]
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for rep in range(3):
            for a, o, b in zip(acts, outs, bufs):
                step(a, o, b)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    for i, (o, ref) in enumerate(zip(outs, alone)):
        assert torch.equal(o, ref), f"step {i} differs when enqueued behind another step"
        assert torch.equal(bufs[i]["counts"], counts_alone[i])
    ctx.close()


def test_decode_step_replays_from_a_cuda_graph():
    """D retains stable graph addresses: a captured D step replays with new inputs written into the same
    tensors and gives the bits of the eager step, with a P context busy on another stream or idle."""
    shape = wl.LayerShape("t", T=48, H=512, E=16, k=4, I=256, shared_I=128, select_bias=True)
    w = wl.make_weights(shape, 1, DEV)
    a1, a2 = wl.make_activations(shape, 2, DEV), wl.make_activations(shape, 3, DEV)
    sd, sp = torch.cuda.Stream(), torch.cuda.Stream()
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 48, B.MOE_PHASE_DECODE), stream=sd)
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    eager1, _ = d.layer(a1["x"], a1["logits"], a1["bias"], *wargs)
    eager2, _ = d.layer(a2["x"], a2["logits"], a2["bias"], *wargs)
    torch.cuda.synchronize()
    # static inputs/outputs of the graph
    x, logits, bias = a1["x"].clone(), a1["logits"].clone(), a1["bias"].clone()
    bufs = B.alloc_step_buffers(48, 4, 16, DEV)
    out = torch.empty(48, 512, dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=sd):
        d.layer(x, logits, bias, *wargs, out=out, bufs=bufs)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager1)
    # new inputs in place, and a P context hammering the GPU meanwhile
    pshape = shape.with_tokens(1024)
    ap = wl.make_activations(pshape, 4, DEV)
    p = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 1024, B.MOE_PHASE_PREFILL), stream=sp)
    x.copy_(a2["x"]); logits.copy_(a2["logits"]); bias.copy_(a2["bias"])
    torch.cuda.synchronize()
    for _ in range(3):
        p.layer(ap["x"], ap["logits"], ap["bias"], *wargs)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager2)
    assert d.moe_ctx_status() == B.MOE_OK and p.moe_ctx_status() == B.MOE_OK
    # eager steps still work after a capture
    again, _ = d.layer(a1["x"], a1["logits"], a1["bias"], *wargs)
    torch.cuda.synchronize()
    assert torch.equal(again, eager1)
    del g
    p.close(); d.close()


def test_turnstile_controller_drives_two_contexts_from_two_host_threads():
    """The paper's protocol end to end on one GPU: a P host thread publishes boundaries from the segment hook and
    stops at its permitted endpoint (P1/P2); a D host thread waits for P to stand there (D1), enqueues a D step
    (D2), orders P's next segment after it on the device and moves the endpoint (D4)."""
    import threading
    shape = wl.LayerShape("t", T=48, H=512, E=16, k=4, I=256, shared_I=128)
    pshape = shape.with_tokens(2048)
    w = wl.make_weights(shape, 1, DEV)
    ad, ap = wl.make_activations(shape, 2, DEV), wl.make_activations(pshape, 3, DEV)
    sp, sd = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    d = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 48, B.MOE_PHASE_DECODE), stream=sd)
    p = B.MoeContext(B.make_config(512, 16, 4, 256, 128, 2048, B.MOE_PHASE_PREFILL), stream=sp)
    wargs = (w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"])
    torch.cuda.synchronize()
    d_alone, _ = d.layer(ad["x"], ad["logits"], None, *wargs)
    p_alone, _ = p.layer(ap["x"], ap["logits"], None, *wargs)
    torch.cuda.synchronize()

    ts = B.Turnstile(span=2)
    n_epochs, errors, d_outs, p_outs = 3, [], [], []
    p_done = threading.Event()

    def p_thread():
        try:
            for e in range(n_epochs):
                assert ts.begin_epoch(e) == B.MOE_OK
                assert ts.publish(e, 0, 20000) == B.MOE_OK          # p = 0: a ready D goes first

                def hook(i, n, e=e):
                    if i + 1 < n:
                        st = ts.publish(e, i + 1, 20000)
                        if st != B.MOE_OK:
                            errors.append(("publish", e, i + 1, st))

                p.moe_ctx_set_segments(4, hook)
                out, _ = p.layer(ap["x"], ap["logits"], None, *wargs)
                p_outs.append(out)
                assert ts.task_done(e) == B.MOE_OK
        except Exception as exc:  # noqa: BLE001
            errors.append(repr(exc))
        finally:
            p_done.set()

    def d_thread():
        try:
            while True:
                stop = p_done.is_set()
                st, active = ts.d_enter(20000)
                assert st == B.MOE_OK
                out, _ = d.layer(ad["x"], ad["logits"], None, *wargs)   # D2 (PreD/PostD rendezvous: one rank)
                ev = torch.cuda.Event()
                ev.record(sd)
                sp.wait_event(ev)       # the P segment admitted next runs after this D step on the device
                d_outs.append(out)
                ts.d_release()          # D4
                if stop:
                    return
        except Exception as exc:  # noqa: BLE001
            errors.append(repr(exc))

    tp, td = threading.Thread(target=p_thread), threading.Thread(target=d_thread)
    tp.start(); td.start()
    tp.join(120); td.join(120)
    torch.cuda.synchronize()
    assert not tp.is_alive() and not td.is_alive() and not errors, errors
    assert len(p_outs) == n_epochs and len(d_outs) >= n_epochs * 5   # 10 boundaries per epoch, span 2
    assert all(torch.equal(o, p_alone) for o in p_outs)
    assert all(torch.equal(o, d_alone) for o in d_outs)
    assert p.moe_ctx_status() == B.MOE_OK and d.moe_ctx_status() == B.MOE_OK
    p.moe_ctx_set_segments(0)
    assert ts.destroy() == B.MOE_OK
    p.close(); d.close()


@pytest.mark.parametrize("variant", [B.MOE_GEMM_LARGE_M, B.MOE_GEMM_SMALL_M])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(variant):
    """Failure detection without faulting the GPU: the context is told (on the host) that its GEMM producers
    issue nothing, so the consumers' bounded waits expire (after 20 ms here: a shared GPU is held for
    milliseconds); the kernels return, the status word says MOE_ERR_TIMEOUT (and is cleared by the read), the
    CUDA context is still alive, and with the hook off the very same context computes a correct step again."""
    shape = wl.LayerShape("t", T=64, H=256, E=8, k=2, I=128)
    w, a = wl.make_weights(shape, 1, DEV), wl.make_activations(shape, 2, DEV)
    ctx = B.MoeContext(B.make_config(256, 8, 2, 128, 0, 64, B.MOE_PHASE_PREFILL, gemm_variant=variant), device=DEV)
    torch.cuda.synchronize()
    good, _ = ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    ctx.moe_ctx_set_wait_limit(20_000)
    ctx.moe_ctx_debug_inject_stall(True)
    ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_ERR_TIMEOUT
    assert ctx.moe_ctx_status() == B.MOE_OK          # the read cleared it
    assert float((torch.ones(4, device=DEV) * 2).sum().item()) == 8.0   # the CUDA context is alive
    ctx.moe_ctx_debug_inject_stall(False)
    ctx.moe_ctx_set_wait_limit(0)
    again, _ = ctx.layer(a["x"], a["logits"], None, w["w_gate_up"], w["w_down"])
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK and torch.equal(again, good)
    ctx.close()


@pytest.mark.parametrize("phase,fmt", [(B.MOE_PHASE_PREFILL, B.MOE_WEIGHTS_BF16), (B.MOE_PHASE_DECODE, B.MOE_WEIGHTS_BF16),
                                       (B.MOE_PHASE_PREFILL, B.MOE_WEIGHTS_FP8_E4M3), (B.MOE_PHASE_DECODE, B.MOE_WEIGHTS_FP8_E4M3)])
def test_nothing_is_written_outside_the_workspace_and_the_callers_arrays(phase, fmt):
    """Guard bands of a known pattern on both sides of the workspace and of every array the caller passes must
    survive whole steps (ragged T, shared expert, segments on the prefill side): no kernel writes out of bounds."""
    T, H, E, k, I, Is = 333, 320, 11, 3, 192, 128
    shape = wl.LayerShape("g", T=T, H=H, E=E, k=k, I=I, shared_I=Is, select_bias=True)
    cfg = B.make_config(H, E, k, I, Is, T, phase, weight_format=fmt)
    nbytes = B.moe_ctx_workspace_bytes(cfg)
    guard = 4096
    pattern = 0xA5

    def guarded(n_bytes):
        raw = torch.full((n_bytes + 2 * guard,), pattern, dtype=torch.uint8, device=DEV)
        return raw, raw[guard:guard + n_bytes]

    raw_ws, ws = guarded((nbytes + 255) // 256 * 256)
    N = T * k
    raws = {}
    views = {}
    for name, n_el, dt in (("topk_idx", N, torch.int32), ("topk_w", N, torch.float32), ("counts", E, torch.int32),
                           ("offsets", E + 1, torch.int32), ("perm", N, torch.int32), ("inv_perm", N, torch.int32),
                           ("out", T * H, torch.bfloat16)):
        esz = torch.empty(0, dtype=dt).element_size()
        nb = (n_el * esz + 255) // 256 * 256
        raws[name], v = guarded(nb)
        views[name] = v[:n_el * esz].view(dt)
    bufs = {"topk_idx": views["topk_idx"].view(T, k), "topk_w": views["topk_w"].view(T, k), "counts": views["counts"],
            "offsets": views["offsets"], "perm": views["perm"], "inv_perm": views["inv_perm"]}
    out = views["out"].view(T, H)
    a = wl.make_activations(shape, 5, DEV)
    torch.cuda.synchronize()
    ctx = B.MoeContext(cfg, workspace=ws)
    for seg in (0, 4):
        if phase == B.MOE_PHASE_PREFILL:
            ctx.moe_ctx_set_segments(seg)
        for _ in range(2):  # a decode context visits both of its buffer sets
            if fmt == B.MOE_WEIGHTS_FP8_E4M3:
                ctx.layer_fp8(a["x"], a["logits"], a["bias"], wl.make_weights_fp8(shape, 6, DEV), out=out, bufs=bufs)
            else:
                w = wl.make_weights(shape, 6, DEV)
                ctx.layer(a["x"], a["logits"], a["bias"], w["w_gate_up"], w["w_down"], w["ws_gate_up"], w["ws_down"],
                          out=out, bufs=bufs)
    torch.cuda.synchronize()
    assert ctx.moe_ctx_status() == B.MOE_OK
    for name, raw in [("workspace", raw_ws)] + list(raws.items()):
        assert bool((raw[:guard] == pattern).all()) and bool((raw[-guard:] == pattern).all()), f"{name}: guard band overwritten"
    assert torch.isfinite(out.float()).all()
    ctx.close()
