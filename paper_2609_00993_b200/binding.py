"""Python binding of the C ABI in include/moe_pd.h -- argument marshalling only.

Same names as the C entry points.  Tensors are torch CUDA tensors used for device memory and
streams; every step of the layer runs in the library's kernels.  If the built library is missing
the import of this module's functions fails loudly: there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoe_pd.so")

MOE_PHASE_PREFILL, MOE_PHASE_DECODE = 0, 1
MOE_OK = 0
MOE_ERR_INVALID_ARG, MOE_ERR_CAPACITY, MOE_ERR_STATE, MOE_ERR_UNSUPPORTED = 1, 2, 3, 4
MOE_ERR_CUDA, MOE_ERR_TIMEOUT, MOE_ERR_BAD_INDEX = 5, 6, 7
MOE_GEMM_AUTO, MOE_GEMM_LARGE_M, MOE_GEMM_SMALL_M, MOE_GEMM_VALIDATION = 0, 1, 2, 3
MOE_WEIGHTS_BF16, MOE_WEIGHTS_FP8_E4M3 = 0, 1
MOE_BOUNDARY_YIELD = -1

STATUS_NAMES = {0: "MOE_OK", 1: "MOE_ERR_INVALID_ARG", 2: "MOE_ERR_CAPACITY", 3: "MOE_ERR_STATE",
                4: "MOE_ERR_UNSUPPORTED", 5: "MOE_ERR_CUDA", 6: "MOE_ERR_TIMEOUT", 7: "MOE_ERR_BAD_INDEX"}

# every symbol include/moe_pd.h declares
EXPORTS = ("moe_version", "moe_ctx_workspace_bytes", "moe_ctx_create", "moe_ctx_destroy", "moe_ctx_status",
           "moe_last_error", "moe_route", "moe_dispatch_layout", "moe_grouped_ffn", "moe_grouped_ffn_fp8", "moe_combine",
           "moe_layer_host", "moe_layer_host_submit", "moe_layer_host_wait",
           "moe_ctx_debug_ptrs", "moe_ctx_debug_ptrs_fp8", "moe_ctx_launch_count", "moe_ctx_set_profiling", "moe_ctx_read_profile",
           "moe_dispatch_layout_static", "moe_ctx_set_segments", "moe_ctx_abandon_step", "moe_turnstile_create", "moe_turnstile_destroy",
           "moe_turnstile_set_span", "moe_turnstile_begin_epoch", "moe_turnstile_publish", "moe_turnstile_task_done",
           "moe_turnstile_d_enter", "moe_turnstile_d_release", "moe_turnstile_state", "moe_ctx_set_wait_limit",
           "moe_ctx_debug_inject_stall", "moe_dispatch_notify", "moe_dispatch_move", "moe_ctx_pending_dispatch",
           "moe_ctx_set_preemption", "moe_ctx_request_yield", "moe_ctx_yield_count")

BOUNDARY_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32)

STAGE_NAMES = ("route", "layout", "permute", "gemm1_swiglu", "gemm2", "shared_gemm1_swiglu", "shared_gemm2", "combine",
               "quantize_x", "quantize_act")


class moe_config(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int32), ("n_experts", ctypes.c_int32), ("top_k", ctypes.c_int32),
                ("inter", ctypes.c_int32), ("n_shared", ctypes.c_int32), ("shared_inter", ctypes.c_int32),
                ("max_tokens", ctypes.c_int32), ("phase", ctypes.c_int32), ("sm_budget", ctypes.c_int32),
                ("gemm_variant", ctypes.c_int32), ("row_gather", ctypes.c_int32), ("routed_scale", ctypes.c_float),
                ("weight_format", ctypes.c_int32)]


class moe_stage_times(ctypes.Structure):
    _fields_ = [("ms", ctypes.c_double * 10), ("calls", ctypes.c_int64 * 10)]


class MoeError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libmoe_pd.so (built in-tree by paper_2609_00993_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_00993_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    cfgp = ctypes.POINTER(moe_config)
    lib.moe_version.restype = ctypes.c_char_p
    lib.moe_version.argtypes = []
    lib.moe_ctx_workspace_bytes.restype = sz
    lib.moe_ctx_workspace_bytes.argtypes = [cfgp]
    lib.moe_ctx_create.restype = i32
    lib.moe_ctx_create.argtypes = [cfgp, vp, sz, vp, ctypes.POINTER(vp)]
    lib.moe_ctx_destroy.restype = i32
    lib.moe_ctx_destroy.argtypes = [vp]
    lib.moe_ctx_status.restype = i32
    lib.moe_ctx_status.argtypes = [vp, ctypes.POINTER(i32)]
    lib.moe_last_error.restype = ctypes.c_char_p
    lib.moe_last_error.argtypes = [vp]
    lib.moe_route.restype = i32
    lib.moe_route.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.moe_dispatch_layout.restype = i32
    lib.moe_dispatch_layout.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    lib.moe_grouped_ffn.restype = i32
    lib.moe_grouped_ffn.argtypes = [vp, vp, vp, vp, vp, vp, i32]
    lib.moe_ctx_debug_ptrs_fp8.restype = i32
    lib.moe_ctx_debug_ptrs_fp8.argtypes = [vp] + [ctypes.POINTER(vp)] * 4
    lib.moe_grouped_ffn_fp8.restype = i32
    lib.moe_grouped_ffn_fp8.argtypes = [vp] * 9 + [i32]
    lib.moe_combine.restype = i32
    lib.moe_combine.argtypes = [vp, vp, vp, i32, vp]
    lib.moe_layer_host.restype = i32
    lib.moe_layer_host.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.moe_layer_host_submit.restype = i32
    lib.moe_layer_host_submit.argtypes = [vp, i32, vp, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.moe_layer_host_wait.restype = i32
    lib.moe_layer_host_wait.argtypes = [vp, i32]
    lib.moe_ctx_debug_ptrs.restype = i32
    lib.moe_ctx_debug_ptrs.argtypes = [vp] + [ctypes.POINTER(vp)] * 6
    lib.moe_ctx_abandon_step.restype = i32
    lib.moe_ctx_abandon_step.argtypes = [vp]
    lib.moe_ctx_launch_count.restype = i64
    lib.moe_ctx_launch_count.argtypes = [vp]
    lib.moe_ctx_set_profiling.restype = i32
    lib.moe_ctx_set_profiling.argtypes = [vp, i32]
    lib.moe_ctx_read_profile.restype = i32
    lib.moe_ctx_read_profile.argtypes = [vp, ctypes.POINTER(moe_stage_times)]
    for name, args in (("moe_turnstile_create", [i32, ctypes.POINTER(vp)]), ("moe_turnstile_destroy", [vp]),
                       ("moe_turnstile_set_span", [vp, i32]), ("moe_turnstile_begin_epoch", [vp, i64, i32]),
                       ("moe_turnstile_publish", [vp, i64, i32, i32]), ("moe_turnstile_task_done", [vp, i64]),
                       ("moe_turnstile_d_enter", [vp, i32, ctypes.POINTER(i32)]), ("moe_turnstile_d_release", [vp]),
                       ("moe_turnstile_state", [vp, ctypes.POINTER(i64)] + [ctypes.POINTER(i32)] * 4)):
        getattr(lib, name).restype = i32
        getattr(lib, name).argtypes = args
    lib.moe_ctx_set_preemption.restype = i32
    lib.moe_ctx_set_preemption.argtypes = [vp, i32]
    lib.moe_ctx_request_yield.restype = i32
    lib.moe_ctx_request_yield.argtypes = [vp, i32]
    lib.moe_ctx_yield_count.restype = i64
    lib.moe_ctx_yield_count.argtypes = [vp]
    lib.moe_dispatch_notify.restype = i32
    lib.moe_dispatch_notify.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.moe_dispatch_move.restype = i32
    lib.moe_dispatch_move.argtypes = [vp, vp]
    lib.moe_ctx_pending_dispatch.restype = i32
    lib.moe_ctx_pending_dispatch.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.moe_ctx_set_wait_limit.restype = i32
    lib.moe_ctx_set_wait_limit.argtypes = [vp, i64]
    lib.moe_ctx_debug_inject_stall.restype = i32
    lib.moe_ctx_debug_inject_stall.argtypes = [vp, i32]
    lib.moe_ctx_set_segments.restype = i32
    lib.moe_ctx_set_segments.argtypes = [vp, i32, BOUNDARY_FN, vp]
    lib.moe_dispatch_layout_static.restype = i32
    lib.moe_dispatch_layout_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    _lib = lib
    return lib


def moe_version() -> str:
    return load_library().moe_version().decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _dev(t: Optional[torch.Tensor], dtype, name):
    if t is None:
        return
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")


def make_config(hidden, n_experts, top_k, inter, shared_inter=0, max_tokens=1, phase=MOE_PHASE_PREFILL, sm_budget=0,
                gemm_variant=MOE_GEMM_AUTO, routed_scale=1.0, row_gather=0, weight_format=MOE_WEIGHTS_BF16) -> moe_config:
    return moe_config(hidden, n_experts, top_k, inter, 1 if shared_inter else 0, shared_inter, max_tokens, phase,
                      sm_budget, gemm_variant, row_gather, routed_scale, weight_format)


def moe_ctx_workspace_bytes(cfg: moe_config) -> int:
    return int(load_library().moe_ctx_workspace_bytes(ctypes.byref(cfg)))


class MoeContext:
    """One phase context (`moe_ctx`).  The workspace is a torch allocation the context keeps alive;
    `stream` is the torch CUDA stream all its calls enqueue on."""

    def __init__(self, cfg: moe_config, stream: Optional[torch.cuda.Stream] = None, device="cuda",
                 workspace: Optional[torch.Tensor] = None):
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = moe_ctx_workspace_bytes(cfg)
        if nbytes == 0:
            raise MoeError(MOE_ERR_INVALID_ARG, "invalid configuration")
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self.workspace = workspace if workspace is not None else torch.empty(nbytes, dtype=torch.uint8,
                                                                                 device=self.device)
            # torch hands out the block on the CURRENT stream and may have recycled it from tensors whose last
            # kernels are still queued there; the context's stream must not touch it before they are done
            self.stream.wait_stream(torch.cuda.current_stream(self.device))
        self.workspace_bytes = nbytes
        handle = ctypes.c_void_p()
        st = self.lib.moe_ctx_create(ctypes.byref(cfg), ctypes.c_void_p(self.workspace.data_ptr()),
                                     self.workspace.numel(), ctypes.c_void_p(self.stream.cuda_stream),
                                     ctypes.byref(handle))
        if st != MOE_OK:
            raise MoeError(st, self.lib.moe_last_error(None).decode())
        self.handle = handle

    # -- plumbing
    def _check(self, st: int):
        if st != MOE_OK:
            raise MoeError(st, self.lib.moe_last_error(self.handle).decode())

    def destroy(self):
        if self.handle is not None:
            self._check(self.lib.moe_ctx_destroy(self.handle))
            self.handle = None

    def close(self):
        """Drain the stream, then destroy."""
        if self.handle is not None:
            self.stream.synchronize()
            self.destroy()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C entry points, same names
    def moe_layer_host_submit(self, slot, logits_host, select_bias, x_host, w_gate_up, w_down, ws_gate_up, ws_down,
                              out_host, T=None):
        """Pipelined form of moe_layer_host: returns once the copies and kernels of the step are enqueued; the
        host tensors (pinned) must stay untouched until moe_layer_host_wait(slot)."""
        for n, t in (("logits_host", logits_host), ("x_host", x_host), ("out_host", out_host)):
            if t.is_cuda:
                raise ValueError(f"{n} must be a host tensor")
        T = x_host.shape[0] if T is None else T
        self._check(self.lib.moe_layer_host_submit(self.handle, slot, _ptr(logits_host), _ptr(select_bias),
                                                   _ptr(x_host), T, _ptr(w_gate_up), _ptr(w_down), _ptr(ws_gate_up),
                                                   _ptr(ws_down), _ptr(out_host)))

    def moe_layer_host_wait(self, slot):
        self._check(self.lib.moe_layer_host_wait(self.handle, slot))

    def moe_ctx_status(self) -> int:
        v = ctypes.c_int32(0)
        self._check(self.lib.moe_ctx_status(self.handle, ctypes.byref(v)))
        return int(v.value)

    def moe_ctx_abandon_step(self):
        self._check(self.lib.moe_ctx_abandon_step(self.handle))

    def moe_ctx_set_preemption(self, enabled: bool):
        self._check(self.lib.moe_ctx_set_preemption(self.handle, int(bool(enabled))))

    def moe_ctx_request_yield(self, on: bool) -> int:
        """Callable from any host thread; returns the status code instead of raising."""
        return int(self.lib.moe_ctx_request_yield(self.handle, int(bool(on))))

    def moe_ctx_yield_count(self) -> int:
        return int(self.lib.moe_ctx_yield_count(self.handle))

    def moe_ctx_set_wait_limit(self, limit_us: int):
        self._check(self.lib.moe_ctx_set_wait_limit(self.handle, int(limit_us)))

    def moe_ctx_debug_inject_stall(self, enabled: bool):
        self._check(self.lib.moe_ctx_debug_inject_stall(self.handle, int(bool(enabled))))

    def moe_ctx_launch_count(self) -> int:
        return int(self.lib.moe_ctx_launch_count(self.handle))

    def moe_ctx_set_segments(self, experts_per_segment: int, fn=None):
        """fn(boundary, n_boundaries) is called on the host after each P segment has been enqueued."""
        if fn is None:
            self._boundary_cb = ctypes.cast(None, BOUNDARY_FN)
        else:
            self._boundary_cb = BOUNDARY_FN(lambda _user, i, n: fn(i, n))  # kept alive by the context
        self._check(self.lib.moe_ctx_set_segments(self.handle, experts_per_segment, self._boundary_cb, None))

    def moe_ctx_set_profiling(self, enabled: bool):
        self._check(self.lib.moe_ctx_set_profiling(self.handle, int(bool(enabled))))

    def moe_ctx_read_profile(self) -> dict:
        """{stage name: (summed device ms, bracketed launches)} since the last read; synchronises the stream."""
        t = moe_stage_times()
        self._check(self.lib.moe_ctx_read_profile(self.handle, ctypes.byref(t)))
        return {n: (float(t.ms[i]), int(t.calls[i])) for i, n in enumerate(STAGE_NAMES)}

    def moe_route(self, logits, select_bias, topk_idx, topk_w, T=None):
        _dev(logits, torch.float32, "logits"); _dev(select_bias, torch.float32, "select_bias")
        _dev(topk_idx, torch.int32, "topk_idx"); _dev(topk_w, torch.float32, "topk_w")
        T = logits.shape[0] if T is None else T
        self._check(self.lib.moe_route(self.handle, _ptr(logits), _ptr(select_bias), T, _ptr(topk_idx), _ptr(topk_w)))

    def moe_dispatch_layout(self, topk_idx, x, counts=None, offsets=None, perm=None, inv_perm=None, T=None):
        _dev(topk_idx, torch.int32, "topk_idx"); _dev(x, torch.bfloat16, "x")
        for n, t in (("counts", counts), ("offsets", offsets), ("perm", perm), ("inv_perm", inv_perm)):
            _dev(t, torch.int32, n)
        T = topk_idx.shape[0] if T is None else T
        self._check(self.lib.moe_dispatch_layout(self.handle, _ptr(topk_idx), T, _ptr(x), _ptr(counts), _ptr(offsets),
                                                 _ptr(perm), _ptr(inv_perm)))

    def moe_dispatch_notify(self, topk_idx, counts=None, offsets=None, perm=None, inv_perm=None, T=None):
        """First half of a split dispatch (counts, scan, permutation); the context then holds a pending dispatch."""
        _dev(topk_idx, torch.int32, "topk_idx")
        for n, t in (("counts", counts), ("offsets", offsets), ("perm", perm), ("inv_perm", inv_perm)):
            _dev(t, torch.int32, n)
        T = topk_idx.shape[0] if T is None else T
        self._check(self.lib.moe_dispatch_notify(self.handle, _ptr(topk_idx), T, _ptr(counts), _ptr(offsets),
                                                 _ptr(perm), _ptr(inv_perm)))

    def moe_dispatch_move(self, x):
        """Second half: the routed data movement of the pending dispatch."""
        _dev(x, torch.bfloat16, "x")
        self._check(self.lib.moe_dispatch_move(self.handle, _ptr(x)))

    def moe_ctx_pending_dispatch(self) -> dict:
        p, t, d = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
        self._check(self.lib.moe_ctx_pending_dispatch(self.handle, ctypes.byref(p), ctypes.byref(t), ctypes.byref(d)))
        return {"pending": bool(p.value), "tokens": int(t.value), "notified_done": bool(d.value)}

    def moe_grouped_ffn(self, w_gate_up, w_down, x, ws_gate_up=None, ws_down=None, T=None):
        for n, t in (("w_gate_up", w_gate_up), ("w_down", w_down), ("x", x), ("ws_gate_up", ws_gate_up),
                     ("ws_down", ws_down)):
            _dev(t, torch.bfloat16, n)
        T = x.shape[0] if T is None else T
        self._check(self.lib.moe_grouped_ffn(self.handle, _ptr(w_gate_up), _ptr(w_down), _ptr(x), _ptr(ws_gate_up),
                                             _ptr(ws_down), T))

    def moe_grouped_ffn_fp8(self, wq_gate_up, sw_gate_up, wq_down, sw_down, wsq_gate_up=None, sws_gate_up=None,
                            wsq_down=None, sws_down=None, T=None):
        """wq_* are uint8 tensors of E4M3 codes, sw_* fp32 per-output-channel scales."""
        for n, t in (("wq_gate_up", wq_gate_up), ("wq_down", wq_down), ("wsq_gate_up", wsq_gate_up),
                     ("wsq_down", wsq_down)):
            _dev(t, torch.uint8, n)
        for n, t in (("sw_gate_up", sw_gate_up), ("sw_down", sw_down), ("sws_gate_up", sws_gate_up),
                     ("sws_down", sws_down)):
            _dev(t, torch.float32, n)
        if T is None:
            raise ValueError("T is required")
        self._check(self.lib.moe_grouped_ffn_fp8(self.handle, _ptr(wq_gate_up), _ptr(sw_gate_up), _ptr(wq_down),
                                                 _ptr(sw_down), _ptr(wsq_gate_up), _ptr(sws_gate_up), _ptr(wsq_down),
                                                 _ptr(sws_down), T))

    def moe_combine(self, topk_w, inv_perm, out, T=None):
        _dev(topk_w, torch.float32, "topk_w"); _dev(inv_perm, torch.int32, "inv_perm"); _dev(out, torch.bfloat16, "out")
        T = out.shape[0] if T is None else T
        self._check(self.lib.moe_combine(self.handle, _ptr(topk_w), _ptr(inv_perm), T, _ptr(out)))

    def moe_layer_host(self, logits_host, select_bias, x_host, w_gate_up, w_down, ws_gate_up, ws_down, out_host,
                       T=None):
        """logits_host / x_host / out_host are HOST tensors (pinned recommended); the rest are device tensors."""
        for n, t in (("logits_host", logits_host), ("x_host", x_host), ("out_host", out_host)):
            if t.is_cuda:
                raise ValueError(f"{n} must be a host tensor")
        T = x_host.shape[0] if T is None else T
        self._check(self.lib.moe_layer_host(self.handle, _ptr(logits_host), _ptr(select_bias), _ptr(x_host), T,
                                            _ptr(w_gate_up), _ptr(w_down), _ptr(ws_gate_up), _ptr(ws_down),
                                            _ptr(out_host)))

    def moe_ctx_debug_ptrs(self) -> dict:
        """Views (no copies) of the workspace buffers of the step in progress / last finished step."""
        ptrs = [ctypes.c_void_p() for _ in range(6)]
        self._check(self.lib.moe_ctx_debug_ptrs(self.handle, *[ctypes.byref(p) for p in ptrs]))
        c = self.cfg
        N = c.max_tokens * c.top_k
        base = self.workspace.data_ptr()

        def view(p, rows, cols, dtype):
            if not p.value or rows * cols == 0:
                return None
            esz = torch.empty(0, dtype=dtype).element_size()
            off = p.value - base
            return self.workspace[off:off + rows * cols * esz].view(dtype).view(rows, cols)

        fp8 = c.weight_format == MOE_WEIGHTS_FP8_E4M3  # such a context keeps no bf16 x_perm
        return {"x_perm": None if fp8 else view(ptrs[0], N, c.hidden, torch.bfloat16), "act": view(ptrs[1], N, c.inter, torch.bfloat16),
                "y_perm": view(ptrs[2], N, c.hidden, torch.bfloat16),
                "y_shared": view(ptrs[3], c.max_tokens, c.hidden, torch.bfloat16) if c.n_shared else None,
                "counts": view(ptrs[4], 1, c.n_experts, torch.int32), "offsets": view(ptrs[5], 1, c.n_experts + 1, torch.int32)}

    def fp8_debug_view(self, name: str, shape, dtype):
        """View of one FP8 buffer of the last step: name in xq, sx, aq, sa."""
        ptrs = [ctypes.c_void_p() for _ in range(4)]
        self._check(self.lib.moe_ctx_debug_ptrs_fp8(self.handle, *[ctypes.byref(p) for p in ptrs]))
        p = ptrs[("xq", "sx", "aq", "sa").index(name)]
        n = 1
        for d in shape:
            n *= d
        esz = torch.empty(0, dtype=dtype).element_size()
        off = p.value - self.workspace.data_ptr()
        return self.workspace[off:off + n * esz].view(dtype).view(*shape)

    def _step_tensors(self, T, k, E, device, bufs, out):
        """Allocates the step's arrays and output when the caller passes none.  torch allocates on its current
        stream; when the context runs on another one, that stream first waits for the current one (a recycled
        block may still be written there) and the tensors are marked as in use on the context's stream."""
        fresh = []
        if bufs is None:
            bufs = alloc_step_buffers(T, k, E, device)
            fresh += list(bufs.values())
        if out is None:
            out = torch.empty(T, self.cfg.hidden, dtype=torch.bfloat16, device=device)
            fresh.append(out)
        cur = torch.cuda.current_stream(self.device)
        if fresh and cur != self.stream:
            self.stream.wait_stream(cur)
            for t in fresh:
                t.record_stream(self.stream)
        return bufs, out

    # -- convenience: one whole step on device tensors (calls the four entry points in order)
    def layer(self, x, logits, select_bias, w_gate_up, w_down, ws_gate_up=None, ws_down=None, out=None, bufs=None):
        T, k, E = x.shape[0], self.cfg.top_k, self.cfg.n_experts
        bufs, out = self._step_tensors(T, k, E, x.device, bufs, out)
        self.moe_route(logits, select_bias, bufs["topk_idx"], bufs["topk_w"], T=T)
        self.moe_dispatch_layout(bufs["topk_idx"], x, bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"],
                                 T=T)
        self.moe_grouped_ffn(w_gate_up, w_down, x, ws_gate_up, ws_down, T=T)
        self.moe_combine(bufs["topk_w"], bufs["inv_perm"], out, T=T)
        return out, bufs

    def layer_fp8(self, x, logits, select_bias, w8: dict, out=None, bufs=None):
        """One step with FP8 weights; `w8` holds wq_gate_up, sw_gate_up, wq_down, sw_down and, with a shared
        expert, wsq_gate_up, sws_gate_up, wsq_down, sws_down (see workloads.make_weights_fp8)."""
        T, k, E = x.shape[0], self.cfg.top_k, self.cfg.n_experts
        bufs, out = self._step_tensors(T, k, E, x.device, bufs, out)
        self.moe_route(logits, select_bias, bufs["topk_idx"], bufs["topk_w"], T=T)
        self.moe_dispatch_layout(bufs["topk_idx"], x, bufs["counts"], bufs["offsets"], bufs["perm"], bufs["inv_perm"],
                                 T=T)
        self.moe_grouped_ffn_fp8(w8["wq_gate_up"], w8["sw_gate_up"], w8["wq_down"], w8["sw_down"],
                                 w8.get("wsq_gate_up"), w8.get("sws_gate_up"), w8.get("wsq_down"), w8.get("sws_down"),
                                 T=T)
        self.moe_combine(bufs["topk_w"], bufs["inv_perm"], out, T=T)
        return out, bufs


def alloc_step_buffers(T: int, k: int, E: int, device) -> dict:
    """Caller-owned per-step arrays of the routing and layout stages."""
    n = max(T * k, 4)
    return {"topk_idx": torch.empty(n, dtype=torch.int32, device=device)[:T * k].view(T, k),
            "topk_w": torch.empty(n, dtype=torch.float32, device=device)[:T * k].view(T, k),
            "counts": torch.empty(E, dtype=torch.int32, device=device),
            "offsets": torch.empty(E + 1, dtype=torch.int32, device=device),
            "perm": torch.empty(n, dtype=torch.int32, device=device)[:T * k],
            "inv_perm": torch.empty(n, dtype=torch.int32, device=device)[:T * k]}


def moe_dispatch_layout_static(topk_idx, n_experts, counts, offsets, perm, inv_perm, stream=None, T=None, top_k=None):
    """Layout without a context and without any allocation (see the header): for embedders that cannot
    allocate device memory.  Returns the moe_status code instead of raising, so callers can test limits."""
    lib = load_library()
    T = topk_idx.shape[0] if T is None else T
    top_k = topk_idx.shape[1] if top_k is None else top_k
    for n, t in (("topk_idx", topk_idx), ("counts", counts), ("offsets", offsets), ("perm", perm), ("inv_perm", inv_perm)):
        _dev(t, torch.int32, n)
    s = stream if stream is not None else torch.cuda.current_stream(topk_idx.device)
    with torch.cuda.device(topk_idx.device):
        return int(lib.moe_dispatch_layout_static(_ptr(topk_idx), T, top_k, n_experts, _ptr(counts), _ptr(offsets),
                                                  _ptr(perm), _ptr(inv_perm), ctypes.c_void_p(s.cuda_stream)))


class Turnstile:
    """One rank's segment-turnstile controller (`moe_turnstile`): host-only, no GPU needed.  Methods return the
    moe_status code (MOE_OK, MOE_ERR_STATE for a protocol violation, MOE_ERR_TIMEOUT) instead of raising."""

    def __init__(self, span: int = 1):
        self.lib = load_library()
        h = ctypes.c_void_p()
        st = self.lib.moe_turnstile_create(span, ctypes.byref(h))
        if st != MOE_OK:
            raise MoeError(st, "moe_turnstile_create")
        self.handle = h

    def begin_epoch(self, epoch: int, d_already_enqueued: bool = False) -> int:
        return int(self.lib.moe_turnstile_begin_epoch(self.handle, epoch, int(d_already_enqueued)))

    def publish(self, epoch: int, boundary: int, timeout_ms: int = -1) -> int:
        return int(self.lib.moe_turnstile_publish(self.handle, epoch, boundary, timeout_ms))

    def task_done(self, epoch: int) -> int:
        return int(self.lib.moe_turnstile_task_done(self.handle, epoch))

    def d_enter(self, timeout_ms: int = -1):
        active = ctypes.c_int32(0)
        st = int(self.lib.moe_turnstile_d_enter(self.handle, timeout_ms, ctypes.byref(active)))
        return st, bool(active.value)

    def d_release(self) -> int:
        return int(self.lib.moe_turnstile_d_release(self.handle))

    def set_span(self, span: int) -> int:
        return int(self.lib.moe_turnstile_set_span(self.handle, span))

    def state(self) -> dict:
        e = ctypes.c_int64(0)
        r, p, k, a = (ctypes.c_int32(0) for _ in range(4))
        self.lib.moe_turnstile_state(self.handle, ctypes.byref(e), ctypes.byref(r), ctypes.byref(p), ctypes.byref(k),
                                     ctypes.byref(a))
        return {"epoch": e.value, "reached": r.value, "permit": p.value, "span": k.value, "active": bool(a.value)}

    def destroy(self) -> int:
        st = int(self.lib.moe_turnstile_destroy(self.handle)) if self.handle else MOE_OK
        if st == MOE_OK:
            self.handle = None
        return st
