"""Pins for the CPU oracle: each stage is checked against something other than itself --
brute force, library routines on special cases, closed forms and invariants --
chosen so that a dropped term, a wrong sign or index, or a transposed operand fails one.
The paper prints no worked example of the layer, so there is no paper value to pin to;
tests/golden/ holds a hand-derived one.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_00993_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(t):
    return wl.bits(t.to(torch.bfloat16))


def _rand_layer(T, H, E, k, I, shared_I=0, seed=0, bias=False):
    shape = wl.LayerShape("t", T=T, H=H, E=E, k=k, I=I, shared_I=shared_I, select_bias=bias)
    w = wl.make_weights(shape, seed)
    a = wl.make_activations(shape, seed + 1)
    return shape, w, a


# ------------------------------------------------------------------ bf16 helpers

def test_bf16_conversions_match_torch():
    g = torch.Generator().manual_seed(5)
    v = torch.randn(4096, generator=g) * 3
    v[:8] = torch.tensor([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -2.5])  # ties and edge values
    want = wl.bits(v.to(torch.bfloat16))
    assert np.array_equal(oracle.f32_to_bf16(v.numpy()), want)
    back = oracle.bf16_to_f32(want)
    assert np.array_equal(back, v.to(torch.bfloat16).float().numpy())


# ------------------------------------------------------------------------ route

def _brute_route_idx(logits, bias, k):
    key = logits if bias is None else (logits + bias[None, :]).astype(np.float32)
    out = np.empty((logits.shape[0], k), np.int32)
    for t in range(logits.shape[0]):
        order = sorted(range(logits.shape[1]), key=lambda e: (-float(key[t, e]), e))
        out[t] = order[:k]
    return out


@pytest.mark.parametrize("T,E,k,with_bias", [(33, 8, 2, False), (17, 256, 8, True), (5, 12, 12, False), (9, 40, 1, True)])
def test_route_indices_brute_force(T, E, k, with_bias):
    g = torch.Generator().manual_seed(E * 131 + k)
    logits = torch.randn(T, E, generator=g).numpy()
    bias = (torch.randn(E, generator=g) * 0.5).numpy() if with_bias else None
    idx, w = oracle.route(logits, bias, k)
    assert np.array_equal(idx, _brute_route_idx(logits, bias, k))


def test_route_tie_rule_on_quantised_logits():
    logits = wl.tie_heavy_logits(64, 16, seed=3).numpy()
    idx, _ = oracle.route(logits, None, 4)
    assert np.array_equal(idx, _brute_route_idx(logits, None, 4))
    # invariants: distinct, keys non-increasing, every unselected expert loses (or ties with a larger index)
    for t in range(64):
        sel = idx[t]
        assert len(set(sel.tolist())) == 4
        ks = logits[t, sel]
        assert all(ks[j] >= ks[j + 1] for j in range(3))
        for j in range(3):
            if ks[j] == ks[j + 1]:
                assert sel[j] < sel[j + 1]
        last_key, last_idx = ks[-1], sel[-1]
        for e in range(16):
            if e not in sel:
                assert logits[t, e] < last_key or (logits[t, e] == last_key and e > last_idx)


def test_route_special_cases():
    # all-equal logits -> the k lowest indices, weights exactly 1/k
    idx, w = oracle.route(np.full((3, 10), 0.75, np.float32), None, 4)
    assert np.array_equal(idx, np.tile(np.arange(4, dtype=np.int32), (3, 1)))
    assert np.array_equal(w, np.full((3, 4), 0.25, np.float32))
    # +0.0 and -0.0 tie: the lower index wins
    l = np.array([[-0.0, 0.0, -1.0]], np.float32)
    idx, _ = oracle.route(l, None, 2)
    assert idx.tolist() == [[0, 1]]
    # k = 1 -> weight exactly routed_scale
    g = torch.Generator().manual_seed(1)
    l = torch.randn(7, 9, generator=g).numpy()
    idx, w = oracle.route(l, None, 1, routed_scale=2.5)
    assert np.array_equal(idx[:, 0], l.argmax(1)) and np.all(w == np.float32(2.5))
    # non-finite input is rejected
    l[0, 0] = np.inf
    with pytest.raises(oracle.OracleError):
        oracle.route(l, None, 2)


def test_route_matches_torch_topk_when_tie_free():
    g = torch.Generator().manual_seed(11)
    logits = torch.randn(128, 256, generator=g)
    idx, w = oracle.route(logits.numpy(), None, 8)
    tv, ti = torch.topk(logits, 8, dim=1)  # library routine; inputs are tie-free so its tie rule is not relied on
    assert np.array_equal(idx, ti.numpy().astype(np.int32))
    want = torch.softmax(tv.double(), dim=1).numpy()
    assert np.allclose(w, want, rtol=1e-6, atol=1e-7)


def test_route_weights_closed_forms():
    g = torch.Generator().manual_seed(12)
    logits = torch.randn(50, 6, generator=g)
    # k = 2: w0 = sigmoid(l0 - l1)
    idx, w = oracle.route(logits.numpy(), None, 2)
    l0 = logits.numpy()[np.arange(50), idx[:, 0]].astype(np.float64)
    l1 = logits.numpy()[np.arange(50), idx[:, 1]].astype(np.float64)
    assert np.allclose(w[:, 0], 1.0 / (1.0 + np.exp(-(l0 - l1))), rtol=1e-6)
    assert np.allclose(w.sum(1), 1.0, atol=1e-6)
    # k = E: full softmax (library) in descending order
    idx, w = oracle.route(logits.numpy(), None, 6)
    sm = torch.softmax(logits.double(), dim=1).numpy()
    assert np.allclose(w, np.take_along_axis(sm, idx.astype(np.int64), 1), rtol=1e-6)
    # shift invariance and routed_scale
    idx2, w2 = oracle.route((logits + 3.0).numpy(), None, 6, routed_scale=2.0)
    assert np.array_equal(idx, idx2) and np.allclose(w2, 2.0 * w, rtol=2e-6)


def test_route_bias_selects_but_does_not_weight():
    logits = np.array([[2.0, 1.0, 0.0, -1.0]], np.float32)
    bias = np.array([-5.0, 0.0, 0.0, 3.0], np.float32)  # keys: -3, 1, 0, 2 -> experts 3, 1
    idx, w = oracle.route(logits, bias, 2)
    assert idx.tolist() == [[3, 1]]
    e = np.exp(np.array([-1.0, 1.0]) - 1.0)
    assert np.allclose(w[0], e / e.sum(), rtol=1e-6)  # softmax over the UNBIASED logits -1 and 1


# ----------------------------------------------------------------------- layout

@pytest.mark.parametrize("N,E", [(0, 4), (1, 1), (128, 8), (1024, 256), (4099, 37)])
def test_layout_matches_numpy(N, E):
    rng = np.random.default_rng(N + E)
    idx = rng.integers(0, E, size=N, dtype=np.int32)
    counts, offsets, perm, inv = oracle.layout(idx, E)
    assert np.array_equal(counts, np.bincount(idx, minlength=E))
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(counts)]))
    assert np.array_equal(perm, np.argsort(idx, kind="stable"))
    assert counts.sum() == N and offsets[-1] == N
    assert np.array_equal(np.sort(perm), np.arange(N))
    assert np.array_equal(inv[perm], np.arange(N))
    e_of_p = idx[perm]
    assert np.all(np.diff(e_of_p) >= 0)
    for e in range(E):
        seg = perm[offsets[e]:offsets[e + 1]]
        assert np.all(np.diff(seg) > 0)


def test_layout_rejects_bad_index():
    with pytest.raises(oracle.OracleError):
        oracle.layout(np.array([0, 5, 1], np.int32), 4)
    with pytest.raises(oracle.OracleError):
        oracle.layout(np.array([0, -1], np.int32), 4)


def test_permute_is_a_bit_copy():
    g = torch.Generator().manual_seed(2)
    x = _bf16_bits(torch.randn(16, 24, generator=g))
    logits = torch.randn(16, 5, generator=g).numpy()
    idx, _ = oracle.route(logits, None, 3)
    _, _, perm, inv = oracle.layout(idx, 5)
    xp = oracle.permute(x, perm, 3)
    for f in range(48):
        assert np.array_equal(xp[inv[f]], x[f // 3])


# -------------------------------------------------------------------------- FFN

def _torch_mlp(x, wgu, wd):
    """Dense SwiGLU MLP from library ops in fp64 (gate = first half of the rows)."""
    I = wd.shape[1]
    x, wgu, wd = x.double(), wgu.double(), wd.double()
    return (torch.nn.functional.silu(x @ wgu[:I].T) * (x @ wgu[I:].T)) @ wd.T


def test_ffn_matches_torch_dense_mlp():
    g = torch.Generator().manual_seed(21)
    M, H, I = 7, 48, 80  # H != I so that a transposed operand cannot pass
    x = torch.randn(M, H, generator=g).to(torch.bfloat16)
    wgu = (torch.randn(2 * I, H, generator=g) * 0.2).to(torch.bfloat16)
    wd = (torch.randn(H, I, generator=g) * 0.2).to(torch.bfloat16)
    y, act = oracle.ffn(wl.bits(x), wl.bits(wgu), wl.bits(wd), want_act=True)
    want = _torch_mlp(x, wgu, wd).numpy()
    assert np.allclose(y, want, rtol=1e-6, atol=1e-6)
    want_act = (torch.nn.functional.silu(x.double() @ wgu[:I].double().T) * (x.double() @ wgu[I:].double().T)).numpy()
    assert np.allclose(act, want_act, rtol=1e-6, atol=1e-6)


def test_ffn_brute_force_python_loops():
    g = torch.Generator().manual_seed(22)
    M, H, I = 2, 3, 4
    x = torch.randn(M, H, generator=g).to(torch.bfloat16)
    wgu = torch.randn(2 * I, H, generator=g).to(torch.bfloat16)
    wd = torch.randn(H, I, generator=g).to(torch.bfloat16)
    y = oracle.ffn(wl.bits(x), wl.bits(wgu), wl.bits(wd))
    xf, wf, df = x.double().tolist(), wgu.double().tolist(), wd.double().tolist()
    for r in range(M):
        a = []
        for i in range(I):
            gi = sum(xf[r][h] * wf[i][h] for h in range(H))
            ui = sum(xf[r][h] * wf[I + i][h] for h in range(H))
            a.append(gi / (1.0 + math.exp(-gi)) * ui)
        for c in range(H):
            assert y[r, c] == pytest.approx(sum(a[i] * df[c][i] for i in range(I)), rel=1e-6, abs=1e-6)


def test_ffn_exact_special_cases():
    g = torch.Generator().manual_seed(23)
    M, H, I = 3, 8, 6
    x = torch.randn(M, H, generator=g).to(torch.bfloat16)
    wgu = torch.randn(2 * I, H, generator=g).to(torch.bfloat16)
    wd = torch.randn(H, I, generator=g).to(torch.bfloat16)
    z = torch.zeros_like
    # zero up, zero gate, zero x -> exactly zero
    wgu0 = wgu.clone(); wgu0[I:] = 0
    assert np.all(oracle.ffn(wl.bits(x), wl.bits(wgu0), wl.bits(wd)) == 0)
    wgu0 = wgu.clone(); wgu0[:I] = 0
    assert np.all(oracle.ffn(wl.bits(x), wl.bits(wgu0), wl.bits(wd)) == 0)
    assert np.all(oracle.ffn(wl.bits(z(x)), wl.bits(wgu), wl.bits(wd)) == 0)
    # one-hot rows of W_down select entries of the activation
    sel = torch.zeros(H, I); sel[torch.arange(H), torch.arange(H) % I] = 1
    y, act = oracle.ffn(wl.bits(x), wl.bits(wgu), _bf16_bits(sel), want_act=True)
    assert np.array_equal(y, act[:, np.arange(H) % I])
    # W_down * 2 -> y * 2 exactly (power of two)
    y1 = oracle.ffn(wl.bits(x), wl.bits(wgu), wl.bits(wd))
    y2 = oracle.ffn(wl.bits(x), wl.bits(wgu), wl.bits((wd.float() * 2).to(torch.bfloat16)))
    assert np.array_equal(y2, 2 * y1)
    # swapping the gate and up halves changes the result (silu is not symmetric)
    swapped = torch.cat([wgu[I:], wgu[:I]])
    assert not np.allclose(oracle.ffn(wl.bits(x), wl.bits(swapped), wl.bits(wd)), y1)


def test_ffn_emulate_bf16_rounds_where_a_bf16_pipeline_stores():
    shape, w, a = _rand_layer(T=5, H=32, E=1, k=1, I=24, seed=4)
    y, act = oracle.ffn(wl.bits(a["x"]), wl.bits(w["w_gate_up"][0]), wl.bits(w["w_down"][0]), emulate_bf16=True,
                        want_act=True)
    for arr in (y, act):
        assert np.array_equal(oracle.bf16_to_f32(oracle.f32_to_bf16(arr)), arr)
    y_ref = oracle.ffn(wl.bits(a["x"]), wl.bits(w["w_gate_up"][0]), wl.bits(w["w_down"][0]))
    assert np.allclose(y, y_ref, rtol=2e-2, atol=1e-4) and not np.array_equal(y, y_ref)


# ------------------------------------------------------------------ whole layer

def _layer(shape, w, a, **kw):
    return oracle.layer(wl.bits(a["x"]), a["logits"].numpy(), None if a["bias"] is None else a["bias"].numpy(), shape.k,
                        wl.bits(w["w_gate_up"]), wl.bits(w["w_down"]),
                        None if w["ws_gate_up"] is None else wl.bits(w["ws_gate_up"]),
                        None if w["ws_down"] is None else wl.bits(w["ws_down"]), **kw)


def test_layer_dense_gate_brute_force():
    """out[t] = sum_e G[t,e] * FFN_e(x[t]) + FFN_shared(x[t]) with every expert evaluated on every token."""
    shape, w, a = _rand_layer(T=12, H=40, E=6, k=3, I=24, shared_I=16, seed=31, bias=True)
    r = _layer(shape, w, a)
    x = a["x"]
    dense = torch.stack([_torch_mlp(x, w["w_gate_up"][e], w["w_down"][e]) for e in range(shape.E)], 1)  # [T,E,H]
    key = a["logits"] + a["bias"][None, :]
    ti = torch.topk(key, shape.k, dim=1).indices
    sel = torch.gather(a["logits"], 1, ti).double()
    G = torch.zeros(shape.T, shape.E, dtype=torch.float64).scatter_(1, ti, torch.softmax(sel, 1))
    want = torch.einsum("te,teh->th", G, dense) + _torch_mlp(x, w["ws_gate_up"], w["ws_down"])
    assert np.allclose(r["out"], want.numpy(), rtol=1e-5, atol=1e-6)
    assert np.allclose(G.sum(1).numpy(), 1.0)


def test_layer_identical_experts_collapse_to_dense_mlp():
    shape, w, a = _rand_layer(T=20, H=32, E=5, k=2, I=48, seed=32)
    w["w_gate_up"][:] = w["w_gate_up"][0]
    w["w_down"][:] = w["w_down"][0]
    r = _layer(shape, w, a)
    want = _torch_mlp(a["x"], w["w_gate_up"][0], w["w_down"][0]).numpy()
    assert np.allclose(r["out"], want, rtol=1e-5, atol=1e-6)


def test_layer_staged_path_equals_definition_path():
    shape, w, a = _rand_layer(T=24, H=64, E=8, k=2, I=32, shared_I=32, seed=33)
    r = _layer(shape, w, a)
    toks = [23, 0, 7, 7, 12]
    out, mag = oracle.layer_tokens(wl.bits(a["x"]), r["topk_idx"], r["topk_w"], wl.bits(w["w_gate_up"]),
                                   wl.bits(w["w_down"]), wl.bits(w["ws_gate_up"]), wl.bits(w["ws_down"]), tokens=toks,
                                   want_term_abs=True)
    assert np.allclose(out, r["out"][toks], rtol=1e-6, atol=1e-7)
    assert np.all(mag + 1e-6 >= np.abs(out))


def test_layer_token_permutation_and_expert_relabelling():
    shape, w, a = _rand_layer(T=16, H=32, E=6, k=2, I=16, seed=34)
    base = _layer(shape, w, a)["out"]
    g = torch.Generator().manual_seed(99)
    tp = torch.randperm(shape.T, generator=g)
    a2 = dict(a, x=a["x"][tp].contiguous(), logits=a["logits"][tp].contiguous())
    assert np.allclose(_layer(shape, w, a2)["out"], base[tp.numpy()], rtol=1e-6, atol=1e-7)
    ep = torch.randperm(shape.E, generator=g)  # new expert i is old expert ep[i]
    w3 = dict(w, w_gate_up=w["w_gate_up"][ep].contiguous(), w_down=w["w_down"][ep].contiguous())
    a3 = dict(a, logits=a["logits"][:, ep].contiguous())
    assert np.allclose(_layer(shape, w3, a3)["out"], base, rtol=1e-6, atol=1e-7)


def test_layer_counts_and_weights_invariants():
    shape, w, a = _rand_layer(T=64, H=16, E=8, k=2, I=16, seed=35)
    r = _layer(shape, w, a)
    assert r["counts"].sum() == shape.T * shape.k
    assert np.allclose(r["topk_w"].sum(1), 1.0, atol=1e-6)
    assert np.array_equal(np.sort(r["perm"]), np.arange(shape.N))


def _read_golden(path):
    vals = {}
    with open(path) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, rest = line.split("=", 1)
            vals[name.strip()] = np.array([float(v) for v in rest.split()], np.float64)
    return vals


def test_layer_hand_derived_example():
    """tests/golden/hand_example.txt: 3 tokens, 3 experts, top-2, H=2, I=1, derived by hand from the definition."""
    gold = _read_golden(os.path.join(GOLDEN, "hand_example.txt"))
    x = torch.tensor(gold["x"].reshape(3, 2), dtype=torch.float32)
    logits = gold["logits"].reshape(3, 3).astype(np.float32)
    wgu = torch.tensor(gold["w_gate_up"].reshape(3, 2, 2), dtype=torch.float32)
    wd = torch.tensor(gold["w_down"].reshape(3, 2, 1), dtype=torch.float32)
    r = oracle.layer(_bf16_bits(x), logits, None, 2, _bf16_bits(wgu), _bf16_bits(wd))
    assert np.array_equal(r["topk_idx"].ravel(), gold["topk_idx"].astype(np.int32))
    assert np.allclose(r["topk_w"].ravel(), gold["topk_w"], rtol=1e-6)
    assert np.array_equal(r["counts"], gold["counts"].astype(np.int32))
    assert np.array_equal(r["perm"], gold["perm"].astype(np.int32))
    assert np.allclose(r["out"].ravel(), gold["out"], rtol=1e-6)
    # the same values from the closed forms they were derived from
    sig = lambda z: 1.0 / (1.0 + math.exp(-z))
    s1, s2, sm1 = sig(1.0), 2 * sig(2.0), -sig(-1.0)
    want = [0.5 * (2 * 2 * s1) + 0.5 * (3 * s2), 0.5 * (-2 * s1) + 0.5 * (3 * s2),
            0.5 * sm1 + 0.5 * (0.5 * 2 * s1), 0.5 * sm1,
            sig(1.0) * (2 * s1) + sig(-1.0) * (0.5 * s2), sig(1.0) * (-s1)]
    assert np.allclose(gold["out"], want, rtol=1e-12)
    # the term magnitude A = sum_j |w_j y_j| and the bf16-storage emulation, both from the same hand derivation
    out, mag = oracle.layer_tokens(_bf16_bits(x), r["topk_idx"], r["topk_w"], _bf16_bits(wgu), _bf16_bits(wd),
                                   want_term_abs=True)
    assert np.allclose(out.ravel(), gold["out"], rtol=1e-6)
    assert np.allclose(mag.ravel(), gold["term_abs"], rtol=1e-6)
    want_mag = [0.5 * 4 * s1 + 0.5 * 3 * s2, 0.5 * 2 * s1 + 0.5 * 3 * s2, 0.5 * -sm1 + 0.5 * s1, 0.5 * -sm1,
                sig(1.0) * 2 * s1 + sig(-1.0) * 0.5 * s2, sig(1.0) * s1]
    assert np.allclose(gold["term_abs"], want_mag, rtol=1e-12)
    assert not np.allclose(gold["term_abs"], np.abs(gold["out"]), rtol=1e-3)  # mixed signs: A is not |out|
    emu = oracle.layer_tokens(_bf16_bits(x), r["topk_idx"], r["topk_w"], _bf16_bits(wgu), _bf16_bits(wd),
                              emulate_bf16=True)
    assert np.allclose(emu.ravel(), gold["out_bf16_storage"], rtol=1e-6)
    staged = oracle.layer(_bf16_bits(x), logits, None, 2, _bf16_bits(wgu), _bf16_bits(wd), emulate_bf16=True)
    assert np.allclose(staged["out"].ravel(), gold["out_bf16_storage"], rtol=1e-6)
    assert not np.allclose(gold["out_bf16_storage"], gold["out"], rtol=1e-4)  # the rounding of a bites


def _bf16_round(v):
    """Round to nearest even onto 8 significant bits with torch's own bfloat16 (a library routine)."""
    return float(torch.tensor(v, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).double())


def test_layer_hand_derived_example_with_shared_expert():
    """tests/golden/hand_example_shared.txt: a shared expert, down weights that make an expert output's bf16
    rounding bite, the term magnitude A including |y_shared|, and the bf16-storage emulation of all three."""
    gold = _read_golden(os.path.join(GOLDEN, "hand_example_shared.txt"))
    x = torch.tensor(gold["x"].reshape(2, 2), dtype=torch.float32)
    logits = gold["logits"].reshape(2, 3).astype(np.float32)
    wgu = torch.tensor(gold["w_gate_up"].reshape(3, 2, 2), dtype=torch.float32)
    wd = torch.tensor(gold["w_down"].reshape(3, 2, 1), dtype=torch.float32)
    wsgu = torch.tensor(gold["ws_gate_up"].reshape(2, 2), dtype=torch.float32)
    wsd = torch.tensor(gold["ws_down"].reshape(2, 1), dtype=torch.float32)
    args = (_bf16_bits(x), logits, None, 2, _bf16_bits(wgu), _bf16_bits(wd), _bf16_bits(wsgu), _bf16_bits(wsd))
    r = oracle.layer(*args)
    assert np.array_equal(r["topk_idx"].ravel(), gold["topk_idx"].astype(np.int32))
    assert np.allclose(r["topk_w"].ravel(), gold["topk_w"], rtol=1e-6)
    assert np.allclose(r["out"].ravel(), gold["out"], rtol=1e-6)
    out, mag = oracle.layer_tokens(args[0], r["topk_idx"], r["topk_w"], args[4], args[5], args[6], args[7],
                                   want_term_abs=True)
    assert np.allclose(out.ravel(), gold["out"], rtol=1e-6)
    assert np.allclose(mag.ravel(), gold["term_abs"], rtol=1e-6)
    emu, emag = oracle.layer_tokens(args[0], r["topk_idx"], r["topk_w"], args[4], args[5], args[6], args[7],
                                    emulate_bf16=True, want_term_abs=True)
    assert np.allclose(emu.ravel(), gold["out_bf16_storage"], rtol=1e-6)
    assert np.allclose(emag.ravel(), gold["term_abs_bf16_storage"], rtol=1e-6)
    assert np.allclose(oracle.layer(*args, emulate_bf16=True)["out"].ravel(), gold["out_bf16_storage"], rtol=1e-6)

    # the stored values again, from the closed forms of the derivation (no oracle code involved)
    sig = lambda z: 1.0 / (1.0 + math.exp(-z))
    silu = lambda z: z * sig(z)
    w0 = (sig(1.0), sig(-1.0))

    def rows(rnd):
        ffn = lambda g, u, down: [rnd(rnd(silu(g) * u) * d) for d in down]
        t0 = (w0, ffn(2, 3, (1, 3)), ffn(3, 1, (0.5, -3)), ffn(-1, 2, (-1, 0.5)))
        t1 = ((0.5, 0.5), ffn(2, -1, (3, -1)), ffn(1, 2, (0.5, -3)), ffn(3, -1, (-1, 0.5)))
        out = [w[0] * ya[c] + w[1] * yb[c] + ys[c] for (w, ya, yb, ys) in (t0, t1) for c in range(2)]
        mag = [abs(w[0] * ya[c]) + abs(w[1] * yb[c]) + abs(ys[c]) for (w, ya, yb, ys) in (t0, t1) for c in range(2)]
        return out, mag

    out_x, mag_x = rows(lambda v: v)
    out_r, mag_r = rows(_bf16_round)
    assert np.allclose(gold["out"], out_x, rtol=1e-12) and np.allclose(gold["term_abs"], mag_x, rtol=1e-12)
    assert np.allclose(gold["out_bf16_storage"], out_r, rtol=1e-12)
    assert np.allclose(gold["term_abs_bf16_storage"], mag_r, rtol=1e-12)
    # plausible mistakes in A are far outside the pin: dropped shared term, unweighted terms, doubled
    no_shared = [abs(w0[0] * 3 * silu(2)) + abs(w0[1] * 0.5 * silu(3))]
    assert abs(gold["term_abs"][0] - no_shared[0]) > 0.1
    # y = 3 a is not a power-of-two multiple: the rounding of y bites (15.84375 is a tie and goes to even, 15.875)
    assert _bf16_round(3 * _bf16_round(3 * silu(2))) == 15.875
