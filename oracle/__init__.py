"""CPU oracle for the MoE layer -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``moe_oracle.c`` (plain C, fp64 accumulation).  The
product path never imports this package: only the tests, the smoke check and
the benchmark's ``cpu_baseline`` / reference arm do.  Nothing here touches a
GPU, and nothing here imports the CUDA package.

Arrays cross the wrapper as numpy: bf16 tensors are ``uint16`` bit patterns,
logits / weights / outputs are ``float32``, indices are ``int32``.  Each
function states the stage it follows in ``moe_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")
_lock = threading.Lock()
_lib = None


class OracleError(RuntimeError):
    pass


_ERR = {1: "invalid argument", 2: "non-finite logit or bias", 3: "expert index out of range", 4: "allocation failed"}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math) and return the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-ftree-vectorize", "-mavx2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
                   "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True, capture_output=True, text=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(rc):
    if rc != 0:
        raise OracleError(_ERR.get(rc, f"error {rc}"))


def _c(a, dtype):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


def bf16_to_f32(bits):
    bits = _c(bits, np.uint16)
    out = np.empty(bits.shape, np.float32)
    _load().oracle_bf16_to_f32(_p(bits), ctypes.c_int64(bits.size), _p(out))
    return out


def f32_to_bf16(vals):
    vals = _c(vals, np.float32)
    out = np.empty(vals.shape, np.uint16)
    _load().oracle_f32_to_bf16(_p(vals), ctypes.c_int64(vals.size), _p(out))
    return out


def route(logits, bias, k, routed_scale=1.0):
    """Stage a1: (topk_idx [T,k] int32, topk_w [T,k] fp32)."""
    logits = _c(logits, np.float32)
    bias = _c(bias, np.float32)
    T, E = logits.shape
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float32)
    _chk(_load().oracle_route(_p(logits), _p(bias), ctypes.c_int32(T), ctypes.c_int32(E), ctypes.c_int32(k),
                              ctypes.c_float(routed_scale), _p(idx), _p(w)))
    return idx, w


def layout(topk_idx, E):
    """Stages a2-a4: (counts [E], offsets [E+1], perm [N], inv_perm [N]) int32."""
    topk_idx = _c(topk_idx, np.int32)
    N = topk_idx.size
    counts = np.empty(E, np.int32)
    offsets = np.empty(E + 1, np.int32)
    perm = np.empty(N, np.int32)
    inv = np.empty(N, np.int32)
    _chk(_load().oracle_layout(_p(topk_idx), ctypes.c_int64(N), ctypes.c_int32(E), _p(counts), _p(offsets), _p(perm),
                               _p(inv)))
    return counts, offsets, perm, inv


def permute(x_bits, perm, k):
    """Stage a5: x_perm [N,H] bf16 bits."""
    x_bits = _c(x_bits, np.uint16)
    perm = _c(perm, np.int32)
    H = x_bits.shape[1]
    out = np.empty((perm.size, H), np.uint16)
    _chk(_load().oracle_permute(_p(x_bits), _p(perm), ctypes.c_int64(perm.size), ctypes.c_int32(k), ctypes.c_int32(H),
                                _p(out)))
    return out


def ffn(x_rows_bits, w_gate_up_bits, w_down_bits, emulate_bf16=False, want_act=False):
    """Stages a6+a7 for one expert (or a8, the shared expert): y [M,H] fp32 (and act [M,I])."""
    x_rows_bits = _c(x_rows_bits, np.uint16)
    w_gate_up_bits = _c(w_gate_up_bits, np.uint16)
    w_down_bits = _c(w_down_bits, np.uint16)
    M, H = x_rows_bits.shape
    I = w_down_bits.shape[1]
    assert w_gate_up_bits.shape == (2 * I, H) and w_down_bits.shape == (H, I)
    y = np.empty((M, H), np.float32)
    act = np.empty((M, I), np.float32) if want_act else None
    _chk(_load().oracle_ffn(_p(x_rows_bits), ctypes.c_int64(M), _p(w_gate_up_bits), _p(w_down_bits), ctypes.c_int32(H),
                            ctypes.c_int32(I), ctypes.c_int32(int(emulate_bf16)), _p(act), _p(y)))
    return (y, act) if want_act else y


def grouped_ffn(x_perm_bits, offsets, w_gate_up_bits, w_down_bits, emulate_bf16=False, want_act=False):
    """Stages a6+a7 over all expert segments: y [N,H] fp32 (and act [N,I])."""
    x_perm_bits = _c(x_perm_bits, np.uint16)
    offsets = _c(offsets, np.int32)
    w_gate_up_bits = _c(w_gate_up_bits, np.uint16)
    w_down_bits = _c(w_down_bits, np.uint16)
    N, H = x_perm_bits.shape
    E, H2, I = w_down_bits.shape
    assert H2 == H and w_gate_up_bits.shape == (E, 2 * I, H) and offsets.size == E + 1
    y = np.empty((N, H), np.float32)
    act = np.empty((N, I), np.float32) if want_act else None
    _chk(_load().oracle_grouped_ffn(_p(x_perm_bits), _p(offsets), ctypes.c_int32(E), _p(w_gate_up_bits),
                                    _p(w_down_bits), ctypes.c_int32(H), ctypes.c_int32(I),
                                    ctypes.c_int32(int(emulate_bf16)), _p(act), _p(y)))
    return (y, act) if want_act else y


def combine(y, inv_perm, topk_w, y_shared=None):
    """Stage a9: out [T,H] fp32."""
    y = _c(y, np.float32)
    inv_perm = _c(inv_perm, np.int32)
    topk_w = _c(topk_w, np.float32)
    y_shared = _c(y_shared, np.float32)
    T, k = topk_w.shape
    H = y.shape[1]
    out = np.empty((T, H), np.float32)
    _chk(_load().oracle_combine(_p(y), _p(inv_perm), _p(topk_w), _p(y_shared), ctypes.c_int32(T), ctypes.c_int32(k),
                                ctypes.c_int32(H), _p(out)))
    return out


def layer_tokens(x_bits, topk_idx, topk_w, w_gate_up_bits, w_down_bits, ws_gate_up_bits=None, ws_down_bits=None,
                 tokens=None, emulate_bf16=False, want_term_abs=False):
    """The dense definition for a set of tokens: out [n,H] fp32 (and the term magnitude A [n,H])."""
    x_bits = _c(x_bits, np.uint16)
    topk_idx = _c(topk_idx, np.int32)
    topk_w = _c(topk_w, np.float32)
    w_gate_up_bits = _c(w_gate_up_bits, np.uint16)
    w_down_bits = _c(w_down_bits, np.uint16)
    ws_gate_up_bits = _c(ws_gate_up_bits, np.uint16)
    ws_down_bits = _c(ws_down_bits, np.uint16)
    T, H = x_bits.shape
    k = topk_idx.shape[1]
    E, _, I = w_down_bits.shape
    if tokens is None:
        n = T
        tok = None
    else:
        tok = _c(np.asarray(tokens, dtype=np.int32), np.int32)
        n = tok.size
    Is = 0 if ws_down_bits is None else ws_down_bits.shape[1]
    out = np.empty((n, H), np.float32)
    mag = np.empty((n, H), np.float32) if want_term_abs else None
    _chk(_load().oracle_layer_tokens(_p(x_bits), _p(topk_idx), _p(topk_w), _p(tok), ctypes.c_int32(n),
                                     ctypes.c_int32(k), ctypes.c_int32(E), ctypes.c_int32(H), ctypes.c_int32(I),
                                     _p(w_gate_up_bits), _p(w_down_bits), _p(ws_gate_up_bits), _p(ws_down_bits),
                                     ctypes.c_int32(Is), ctypes.c_int32(int(emulate_bf16)), _p(out), _p(mag)))
    return (out, mag) if want_term_abs else out


def layer(x_bits, logits, bias, k, w_gate_up_bits, w_down_bits, ws_gate_up_bits=None, ws_down_bits=None,
          routed_scale=1.0, emulate_bf16=False):
    """Whole layer through the explicit stages a1..a9, in order.  Returns a dict of every stage's result."""
    E = w_down_bits.shape[0]
    idx, w = route(logits, bias, k, routed_scale)
    counts, offsets, perm, inv = layout(idx, E)
    x_perm = permute(x_bits, perm, k)
    y, act = grouped_ffn(x_perm, offsets, w_gate_up_bits, w_down_bits, emulate_bf16, want_act=True)
    y_sh = None
    if ws_gate_up_bits is not None:
        y_sh = ffn(x_bits, ws_gate_up_bits, ws_down_bits, emulate_bf16)
    out = combine(y, inv, w, y_sh)
    return dict(topk_idx=idx, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv, x_perm=x_perm,
                act=act, y=y, y_shared=y_sh, out=out)


# ----------------------------------------------------------------------------- FP8 precision variant
def e4m3_decode(codes):
    """E4M3 codes (uint8) -> fp32 values."""
    codes = _c(codes, np.uint8)
    out = np.empty(codes.shape, np.float32)
    _load().oracle_e4m3_decode(_p(codes), ctypes.c_int64(codes.size), _p(out))
    return out


def e4m3_encode(vals):
    """fp32 values -> E4M3 codes (round to nearest even, saturating at +-448)."""
    vals = _c(vals, np.float32)
    out = np.empty(vals.shape, np.uint8)
    _load().oracle_e4m3_encode(_p(vals), ctypes.c_int64(vals.size), _p(out))
    return out


def quantize_rows(x_bits):
    """Per-row dynamic quantisation of bf16 rows [M,n]: (codes [M,n] uint8, scale [M] fp32)."""
    x_bits = _c(x_bits, np.uint16)
    M, n = x_bits.shape
    q = np.empty((M, n), np.uint8)
    s = np.empty(M, np.float32)
    _chk(_load().oracle_quantize_rows(_p(x_bits), ctypes.c_int64(M), ctypes.c_int32(n), _p(q), _p(s)))
    return q, s


def gemm1_fp8(xq, sx, wq_gate_up, sw_gate_up):
    """GEMM1 + SwiGLU of the FP8 variant for one expert: act [M,I] bf16 bits."""
    xq, sx = _c(xq, np.uint8), _c(sx, np.float32)
    wq_gate_up, sw_gate_up = _c(wq_gate_up, np.uint8), _c(sw_gate_up, np.float32)
    M, H = xq.shape
    I = wq_gate_up.shape[0] // 2
    assert wq_gate_up.shape == (2 * I, H) and sw_gate_up.shape == (2 * I,) and sx.shape == (M,)
    act = np.empty((M, I), np.uint16)
    _chk(_load().oracle_gemm1_fp8(_p(xq), _p(sx), ctypes.c_int64(M), _p(wq_gate_up), _p(sw_gate_up),
                                  ctypes.c_int32(H), ctypes.c_int32(I), _p(act)))
    return act


def gemm2_fp8(aq, sa, wq_down, sw_down):
    """GEMM2 of the FP8 variant for one expert: y [M,H] fp32."""
    aq, sa = _c(aq, np.uint8), _c(sa, np.float32)
    wq_down, sw_down = _c(wq_down, np.uint8), _c(sw_down, np.float32)
    M, I = aq.shape
    H = wq_down.shape[0]
    assert wq_down.shape == (H, I) and sw_down.shape == (H,) and sa.shape == (M,)
    y = np.empty((M, H), np.float32)
    _chk(_load().oracle_gemm2_fp8(_p(aq), _p(sa), ctypes.c_int64(M), _p(wq_down), _p(sw_down), ctypes.c_int32(H),
                                  ctypes.c_int32(I), _p(y)))
    return y


def ffn_fp8(x_rows_bits, wq_gate_up, sw_gate_up, wq_down, sw_down, want_stages=False):
    """One expert of the FP8 variant on bf16 rows: quantise -> GEMM1 + SwiGLU -> quantise -> GEMM2.
    Returns y [M,H] fp32 (and a dict of the intermediate stages)."""
    xq, sx = quantize_rows(x_rows_bits)
    act = gemm1_fp8(xq, sx, wq_gate_up, sw_gate_up)
    aq, sa = quantize_rows(act)
    y = gemm2_fp8(aq, sa, wq_down, sw_down)
    return (y, dict(xq=xq, sx=sx, act=act, aq=aq, sa=sa)) if want_stages else y


def layer_fp8(x_bits, logits, bias, k, wq_gate_up, sw_gate_up, wq_down, sw_down, wsq_gate_up=None, sws_gate_up=None,
              wsq_down=None, sws_down=None, routed_scale=1.0):
    """Whole layer of the FP8 variant through the explicit stages; routing, layout, row movement and combine are
    the bf16 layer's.  Returns a dict of every stage's result."""
    E = wq_down.shape[0]
    H = x_bits.shape[1]
    idx, w = route(logits, bias, k, routed_scale)
    counts, offsets, perm, inv = layout(idx, E)
    x_perm = permute(x_bits, perm, k)
    y = np.zeros((x_perm.shape[0], H), np.float32)
    act = np.zeros((x_perm.shape[0], wq_down.shape[2]), np.uint16)
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e + 1])
        if r1 > r0:
            y[r0:r1], st = ffn_fp8(x_perm[r0:r1], wq_gate_up[e], sw_gate_up[e], wq_down[e], sw_down[e],
                                   want_stages=True)
            act[r0:r1] = st["act"]
    y_sh = None
    if wsq_gate_up is not None:
        y_sh = ffn_fp8(x_bits, wsq_gate_up, sws_gate_up, wsq_down, sws_down)
    out = combine(y, inv, w, y_sh)
    return dict(topk_idx=idx, topk_w=w, counts=counts, offsets=offsets, perm=perm, inv_perm=inv, x_perm=x_perm,
                act=act, y=y, y_shared=y_sh, out=out)
