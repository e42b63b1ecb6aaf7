"""Shared helpers of the GPU parity tests: move seeded inputs to the host for the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2609_00993_b200 import workloads as wl

# Tolerances of the layer output (bf16) against the oracle's unrounded result:
#   relative L2 error <= 5e-3 everywhere;
#   max abs error <= 2e-2 literally where the outputs are small enough for bf16 to resolve it (C1, C3);
#   at the DeepSeek-V3 shapes outputs reach |v| ~ 10 where half a bf16 ulp is already 0.031, so the bound is
#   applied in its forward-error form |d| <= 2e-2 * (1 + A), A = sum_j |w_j y_j| + |y_shared| (equal to the
#   literal bound as A -> 0).
REL_L2_MAX = 5e-3
MAX_ABS = 2e-2
TOPK_W_ATOL, TOPK_W_RTOL = 1e-6, 1e-5


def np_i32(t):
    return t.detach().cpu().numpy().astype(np.int32, copy=False)


def np_f32(t):
    return t.detach().float().cpu().numpy()


def check_topk_w(gpu_w, ref_w):
    gpu_w, ref_w = np_f32(gpu_w), np.asarray(ref_w)
    assert np.all(np.abs(gpu_w - ref_w) <= TOPK_W_ATOL + TOPK_W_RTOL * np.abs(ref_w)), \
        f"topk_w max err {np.abs(gpu_w - ref_w).max()}"


def layer_errors(out_gpu, out_ref, term_abs=None):
    g = np_f32(out_gpu).astype(np.float64)
    r = np.asarray(out_ref, np.float64)
    d = g - r
    tok_rel = (np.linalg.norm(d, axis=-1) / np.maximum(np.linalg.norm(r, axis=-1), 1e-30)) if d.ndim == 2 and d.size else np.zeros(1)
    res = {"worst_token_rel_l2": float(tok_rel.max()),
           "max_abs": float(np.abs(d).max()) if d.size else 0.0,
           "rel_l2": float(np.linalg.norm(d) / max(np.linalg.norm(r), 1e-30)) if d.size else 0.0,
           "frac_gt": float((np.abs(d) > MAX_ABS).mean()) if d.size else 0.0}
    if term_abs is not None:
        res["scaled_max"] = float((np.abs(d) / (1.0 + np.asarray(term_abs, np.float64))).max()) if d.size else 0.0
    return res


def check_layer(out_gpu, out_ref, term_abs=None, literal=True, label=""):
    e = layer_errors(out_gpu, out_ref, term_abs)
    print(f"[parity {label}] max_abs={e['max_abs']:.4g} rel_l2={e['rel_l2']:.4g} worst token rel_l2={e['worst_token_rel_l2']:.4g} "
          f"frac>2e-2={e['frac_gt']:.3g}"
          + (f" scaled_max={e['scaled_max']:.4g}" if "scaled_max" in e else ""))
    assert e["rel_l2"] <= REL_L2_MAX, f"{label}: rel L2 {e['rel_l2']}"
    assert e["worst_token_rel_l2"] <= REL_L2_MAX, f"{label}: worst token rel L2 {e['worst_token_rel_l2']}"
    if literal:
        assert e["max_abs"] <= MAX_ABS, f"{label}: max abs {e['max_abs']}"
    else:
        assert term_abs is not None
        assert e["scaled_max"] <= MAX_ABS, f"{label}: scaled max abs {e['scaled_max']}"
    return e


def oracle_tokens_from_device(x, topk_idx, topk_w, weights, tokens, want_term_abs=True, emulate_bf16=False):
    """Dense-definition oracle output for `tokens`, pulling only the experts each token uses off the GPU
    (the V3-shaped routed weights are 22.5 GB; no host copy of all of them is ever made)."""
    k = topk_idx.shape[1]
    H = x.shape[1]
    outs, mags = [], []
    ws_gu = None if weights["ws_gate_up"] is None else wl.bits(weights["ws_gate_up"])
    ws_d = None if weights["ws_down"] is None else wl.bits(weights["ws_down"])
    idx_h = np_i32(topk_idx)
    w_h = np_f32(topk_w)
    for t in tokens:
        sel = torch.as_tensor(idx_h[t].astype(np.int64), device=weights["w_gate_up"].device)
        gu = wl.bits(weights["w_gate_up"].index_select(0, sel))
        dn = wl.bits(weights["w_down"].index_select(0, sel))
        xt = wl.bits(x[t:t + 1])
        o, m = oracle.layer_tokens(xt, np.arange(k, dtype=np.int32)[None, :], w_h[t:t + 1], gu, dn, ws_gu, ws_d,
                                   tokens=None, emulate_bf16=emulate_bf16, want_term_abs=True)
        outs.append(o[0])
        mags.append(m[0])
    out = np.stack(outs) if outs else np.zeros((0, H), np.float32)
    mag = np.stack(mags) if mags else np.zeros((0, H), np.float32)
    return (out, mag) if want_term_abs else out


def sample_tokens(T, counts, offsets, perm, k, n, seed=0):
    """Token sample for large configs: random tokens plus the first/last row of the most and the least
    loaded non-empty experts."""
    rng = np.random.default_rng(seed)
    toks = set(rng.choice(T, size=min(n, T), replace=False).tolist())
    nz = np.nonzero(counts)[0]
    if nz.size:
        for e in (nz[np.argmax(counts[nz])], nz[np.argmin(counts[nz])]):
            toks.add(int(perm[offsets[e]] // k))
            toks.add(int(perm[offsets[e + 1] - 1] // k))
    return sorted(toks)


def check_against_storage_precision(out_gpu, out_ref, out_emul, label=""):
    """The GPU result is as accurate as the specified storage precisions allow: its error against the unrounded
    oracle is compared with that of the oracle's own bf16-storage emulation (activation, expert outputs and layer
    output rounded to bf16 where a bf16 pipeline stores them) and with the rounding of the exact result alone."""
    g = np_f32(out_gpu).astype(np.float64)
    r = np.asarray(out_ref, np.float64)
    m = np.asarray(out_emul, np.float64)
    r_bf16 = torch.from_numpy(np.asarray(out_ref, np.float32)).to(torch.bfloat16).double().numpy()
    m_bf16 = torch.from_numpy(np.asarray(out_emul, np.float32)).to(torch.bfloat16).double().numpy()  # + the output's own rounding
    floor_round = float(np.abs(r_bf16 - r).max())
    floor_emul = float(np.abs(m_bf16 - r).max())
    rel_emul = float(np.linalg.norm(m_bf16 - r) / max(np.linalg.norm(r), 1e-30))
    max_abs = float(np.abs(g - r).max())
    rel = float(np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30))
    print(f"[storage floors {label}] gpu max_abs={max_abs:.4g} rel_l2={rel:.4g} | bf16 of the exact result: "
          f"{floor_round:.4g} | bf16-storage emulation: max_abs={floor_emul:.4g} rel_l2={rel_emul:.4g}")
    assert max_abs <= 1.5 * floor_emul, f"{label}: max abs {max_abs} against emulation floor {floor_emul}"
    assert rel <= 1.1 * rel_emul, f"{label}: rel L2 {rel} against emulation {rel_emul}"


def term_abs_from_stages(ref):
    """A[t,c] = sum_j |w[t,j] * y[inv_perm[t,j], c]| + |y_shared[t,c]| from the staged oracle results (the same
    quantity oracle.layer_tokens returns as term_abs, which is pinned to hand-derived values)."""
    w = np.asarray(ref["topk_w"], np.float64)
    T, k = w.shape
    y = np.asarray(ref["y"], np.float64)
    inv = np.asarray(ref["inv_perm"]).reshape(T, k)
    A = np.zeros((T, y.shape[1]))
    for j in range(k):
        A += np.abs(w[:, j:j + 1] * y[inv[:, j]])
    if ref.get("y_shared") is not None:
        A += np.abs(np.asarray(ref["y_shared"], np.float64))
    return A


def check_layer_strict(out_gpu, ref, label=""):
    """Gates for the small whole-layer cases (every token compared): relative L2 over the tensor and for the worst
    token <= 5e-3, and elementwise |d| <= 2^-7 (max A + 1e-3) with A the term magnitude -- three bf16 roundings
    (activation, expert output, layer output) of half an ulp = 2^-9 relative each on terms bounded by A, so a
    wrong element or a wrong short row cannot hide in a whole-tensor norm."""
    e = layer_errors(out_gpu, ref["out"])
    A = term_abs_from_stages(ref)
    bound = 2.0 ** -7 * (float(A.max()) if A.size else 0.0) + 1e-3 * 2.0 ** -7
    assert e["rel_l2"] <= REL_L2_MAX, f"{label}: rel L2 {e}"
    assert e["worst_token_rel_l2"] <= 2 * REL_L2_MAX, f"{label}: worst token rel L2 {e}"
    assert e["max_abs"] <= bound, f"{label}: max abs {e['max_abs']} against {bound}"
    return e


def oracle_tokens_grouped(x, topk_idx, topk_w, weights, tokens, emulate_too=False):
    """Oracle output for many sampled tokens of a large layer.  The experts these tokens use are pulled off the
    GPU one at a time (never all 22.5 GB at once); each expert's FFN runs on all sampled rows routed to it
    (oracle.ffn), and oracle.combine sums them.  Returns out [n,H], term magnitude A [n,H] and, on request, the
    bf16-storage emulation of out."""
    k = topk_idx.shape[1]
    tokens = np.asarray(tokens, np.int64)
    n = tokens.size
    H = x.shape[1]
    idx_h = np_i32(topk_idx)[tokens]          # [n,k]
    w_h = np_f32(topk_w)[tokens]              # [n,k]
    x_rows = wl.bits(x[torch.as_tensor(tokens, device=x.device)])  # [n,H] bits
    y = np.zeros((n * k, H), np.float32)
    y_em = np.zeros((n * k, H), np.float32) if emulate_too else None
    flat_e = idx_h.reshape(-1)
    for e in np.unique(flat_e):
        slots = np.nonzero(flat_e == e)[0]
        gu = wl.bits(weights["w_gate_up"][int(e)])
        dn = wl.bits(weights["w_down"][int(e)])
        rows = np.ascontiguousarray(x_rows[slots // k])
        y[slots] = oracle.ffn(rows, gu, dn)
        if emulate_too:
            y_em[slots] = oracle.ffn(rows, gu, dn, emulate_bf16=True)
    y_sh = y_sh_em = None
    if weights["ws_gate_up"] is not None:
        sgu, sdn = wl.bits(weights["ws_gate_up"]), wl.bits(weights["ws_down"])
        y_sh = oracle.ffn(x_rows, sgu, sdn)
        if emulate_too:
            y_sh_em = oracle.ffn(x_rows, sgu, sdn, emulate_bf16=True)
    inv = np.arange(n * k, dtype=np.int32)
    out = oracle.combine(y, inv, w_h, y_sh)
    A = np.abs(w_h[:, :, None].astype(np.float64) * y.reshape(n, k, H)).sum(1)
    if y_sh is not None:
        A += np.abs(y_sh)
    out_em = oracle.combine(y_em, inv, w_h, y_sh_em) if emulate_too else None
    return out, A, out_em


def sample_tokens_wide(T, counts, offsets, perm, k, n=256, seed=0):
    """At least n tokens of a large batch: random ones plus the first and the last row of a spread of expert
    segments -- the most loaded, the least loaded non-empty, one per class of (rows mod 128) in (0,32], (32,64],
    (64,96], (96,128] (the short last-tile boxes of the large-M kernel), one with 129..256 rows and one with more
    than 256 (single- and multi-chunk tiles of the small-M kernel), and a few random ones."""
    rng = np.random.default_rng(seed)
    toks = set(rng.choice(T, size=min(n, T), replace=False).tolist())
    nz = np.nonzero(counts)[0]
    picks = []
    if nz.size:
        picks += [nz[np.argmax(counts[nz])], nz[np.argmin(counts[nz])]]
        for lo, hi in ((0, 32), (32, 64), (64, 96), (96, 128)):
            m = [e for e in nz if lo < ((counts[e] - 1) % 128) + 1 <= hi]
            picks += m[:1]
        picks += [e for e in nz if 128 < counts[e] <= 256][:1] + [e for e in nz if counts[e] > 256][:1]
        picks += rng.choice(nz, size=min(4, nz.size), replace=False).tolist()
    for e in picks:
        toks.add(int(perm[offsets[e]] // k))
        toks.add(int(perm[offsets[e + 1] - 1] // k))
    return sorted(toks), len(set(int(e) for e in picks))
