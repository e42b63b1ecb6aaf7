"""Pins of the oracle's FP8 (E4M3) precision variant against things other than itself: torch's own float8
type for the codec, brute force over all codes for nearest-even rounding, closed-form properties of the per-row
quantisation, torch float64 matmuls of independently decoded operands for the two GEMMs, and the bf16 oracle
for inputs that E4M3 represents exactly."""
import numpy as np
import torch

import oracle

RNG = np.random.default_rng(8)


def _torch_decode(codes):
    return torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).to(torch.float64)


def _bf16_bits(vals_f32):
    return torch.from_numpy(np.ascontiguousarray(vals_f32, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_decode_matches_torch_float8_for_all_256_codes():
    codes = np.arange(256, dtype=np.uint8)
    mine = oracle.e4m3_decode(codes)
    ref = _torch_decode(codes).numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    assert np.array_equal(mine[~np.isnan(mine)].astype(np.float64), ref[~np.isnan(ref)])
    # format facts: largest finite 448, smallest subnormal 2^-9, first normal 2^-6, only S.1111.111 is NaN
    assert mine[0x7E] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6 and np.isnan(mine[0x7F])
    assert np.isnan(mine).sum() == 2


def test_encode_is_nearest_even_by_brute_force_and_saturates():
    finite = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], np.uint8)
    vals = oracle.e4m3_decode(finite).astype(np.float64)
    x = np.concatenate([RNG.standard_normal(4000) * s for s in (1e-3, 2e-2, 1.0, 40.0, 300.0)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]
    # exact midpoints between neighbouring positive codes: ties must go to the even code
    pos = np.sort(vals[vals >= 0])
    mids = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)
    x = np.concatenate([x, mids, -mids])
    got = oracle.e4m3_encode(x)
    got_val = oracle.e4m3_decode(got).astype(np.float64)
    dist = np.abs(vals[None, :] - x.astype(np.float64)[:, None])
    best = dist.min(axis=1)
    assert np.array_equal(np.abs(got_val - x), best)  # a nearest representable value
    tie = (dist == best[:, None]).sum(axis=1) > 1
    nz = tie & (got_val != 0)
    assert np.all((got[nz] & 1) == 0)  # ties: even mantissa
    assert tie.sum() >= 2 * (len(mids) - 1)
    # the same codes as torch's conversion inside the finite range
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    same = (got == ref) | ((got_val == 0) & (oracle.e4m3_decode(ref) == 0))  # +0 / -0
    assert np.all(same)
    # saturation instead of NaN beyond the range
    big = np.array([448.5, 464.0, 1e4, 3e38, -449.0, -1e9], np.float32)
    assert list(oracle.e4m3_encode(big)) == [0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE]


def test_quantize_rows_scale_codes_and_error_bound():
    x = (RNG.standard_normal((37, 192)) * RNG.choice([1e-2, 1.0, 50.0], (37, 1))).astype(np.float32)
    x[5] = 0.0
    bits = _bf16_bits(x)
    xv = oracle.bf16_to_f32(bits)
    q, s = oracle.quantize_rows(bits)
    amax = np.abs(xv).max(axis=1)
    assert s[5] == np.float32(2.0 ** -100) / np.float32(448.0) and np.all(q[5] == 0)  # the floor of amax
    nzr = amax > 0
    assert np.array_equal(s[nzr], (amax[nzr] / np.float32(448.0)).astype(np.float32))
    dq = oracle.e4m3_decode(q).astype(np.float64)
    assert np.all(np.abs(dq[nzr]).max(axis=1) == 448.0)  # the row's largest element lands on the largest code
    # reconstruction error: half a code step = 2^-4 relative for normal codes, 2^-10 * scale below the normal range
    err = np.abs(dq * s[:, None].astype(np.float64) - xv)
    bound = np.maximum(np.abs(xv) * 2.0 ** -4, s[:, None].astype(np.float64) * 2.0 ** -10) * (1 + 1e-6)
    assert np.all(err <= bound)
    # sign symmetry and invariance of the codes under a power-of-two rescaling of the row
    q2, s2 = oracle.quantize_rows(_bf16_bits(-4.0 * xv))
    assert np.array_equal(q2 & 0x7F, q & 0x7F) and np.array_equal(s2[nzr], 4.0 * s[nzr])
    assert np.array_equal((q2 ^ q)[dq != 0] & 0x80, np.full((dq != 0).sum(), 0x80, np.uint8))


def _rand_codes(shape, sigma=100.0):
    v = torch.from_numpy((RNG.standard_normal(shape) * sigma).astype(np.float32)).clamp(-448, 448)
    return v.to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def test_gemms_match_torch_float64_on_independently_decoded_operands():
    M, H, I = 9, 128, 64
    xq, wq1, wq2 = _rand_codes((M, H)), _rand_codes((2 * I, H)), _rand_codes((H, I))
    sx = RNG.uniform(1e-3, 2e-3, M).astype(np.float32)
    sw1 = RNG.uniform(1e-4, 3e-4, 2 * I).astype(np.float32)
    sw2 = RNG.uniform(1e-4, 3e-4, H).astype(np.float32)
    X, W1, W2 = _torch_decode(xq), _torch_decode(wq1), _torch_decode(wq2)
    z = (X @ W1.T) * torch.from_numpy(sx).double()[:, None] * torch.from_numpy(sw1).double()[None, :]
    g, u = z[:, :I], z[:, I:]
    a_ref = (g / (1 + torch.exp(-g)) * u)
    act = oracle.bf16_to_f32(oracle.gemm1_fp8(xq, sx, wq1, sw1)).astype(np.float64)
    a_np = a_ref.numpy()
    assert np.all(np.abs(act - a_np) <= np.abs(a_np) * 2.0 ** -8 + 1e-30)      # bf16 rounding of the right value
    assert np.mean(act == a_ref.float().to(torch.bfloat16).double().numpy()) > 0.999  # and the same rounding
    aq = _rand_codes((M, I))
    sa = RNG.uniform(1e-3, 2e-3, M).astype(np.float32)
    y = oracle.gemm2_fp8(aq, sa, wq2, sw2).astype(np.float64)
    y_ref = ((_torch_decode(aq) @ W2.T) * torch.from_numpy(sa).double()[:, None]
             * torch.from_numpy(sw2).double()[None, :]).numpy()
    assert np.allclose(y, y_ref, rtol=1e-6, atol=0)
    # a transposed weight operand or swapped gate/up halves would not survive these
    assert not np.allclose(oracle.gemm2_fp8(aq, sa, np.ascontiguousarray(wq2.reshape(I, H).T), sw2), y_ref, rtol=1e-2)
    swapped = np.concatenate([wq1[I:], wq1[:I]])
    act_sw = oracle.bf16_to_f32(oracle.gemm1_fp8(xq, sx, swapped, np.concatenate([sw1[I:], sw1[:I]])))
    assert not np.allclose(act_sw, act, rtol=1e-2)


def test_exactly_representable_inputs_reduce_to_the_bf16_oracle():
    """Rows whose values E4M3 holds exactly and whose largest magnitude is 448 get scale 1 and lossless codes, so
    GEMM1 + SwiGLU of the FP8 variant must reproduce the bf16 oracle's activation for the same numbers."""
    M, H, I = 6, 64, 32
    xq = _rand_codes((M, H), 60.0)
    xq[:, 0] = 0x7E  # amax = 448 -> scale exactly 1
    wq = _rand_codes((2 * I, H), 2.0)
    xv, wv = oracle.e4m3_decode(xq), oracle.e4m3_decode(wq) * np.float32(2.0 ** -12)
    x_bits, w_bits = _bf16_bits(xv), _bf16_bits(wv)
    assert np.array_equal(oracle.bf16_to_f32(x_bits), xv) and np.array_equal(oracle.bf16_to_f32(w_bits), wv)
    q, s = oracle.quantize_rows(x_bits)
    assert np.array_equal(q & 0x7F, xq & 0x7F) and np.all(s == 1.0)
    act8 = oracle.gemm1_fp8(q, s, wq, np.full(2 * I, 2.0 ** -12, np.float32))
    w_down = _bf16_bits(np.zeros((H, I), np.float32))
    _, act16 = oracle.ffn(x_bits, w_bits, w_down, emulate_bf16=True, want_act=True)
    assert np.array_equal(oracle.bf16_to_f32(act8), act16)


def test_fp8_layer_stays_within_the_quantisation_error_of_the_bf16_layer():
    T, H, E, k, I = 48, 128, 4, 2, 64
    x = RNG.standard_normal((T, H)).astype(np.float32)
    logits = RNG.standard_normal((T, E)).astype(np.float32)
    w1 = (RNG.standard_normal((E, 2 * I, H)) / np.sqrt(H)).astype(np.float32)
    w2 = (RNG.standard_normal((E, H, I)) / np.sqrt(I)).astype(np.float32)
    x_bits, w1_bits, w2_bits = _bf16_bits(x), _bf16_bits(w1), _bf16_bits(w2)
    ref = oracle.layer(x_bits, logits, None, k, w1_bits, w2_bits)
    q1, s1 = oracle.quantize_rows(w1_bits.reshape(E * 2 * I, H))   # per-output-channel weight quantisation
    q2, s2 = oracle.quantize_rows(w2_bits.reshape(E * H, I))
    out = oracle.layer_fp8(x_bits, logits, None, k, q1.reshape(E, 2 * I, H), s1.reshape(E, 2 * I),
                           q2.reshape(E, H, I), s2.reshape(E, H))
    for name in ("topk_idx", "perm", "counts"):
        assert np.array_equal(out[name], ref[name])
    rel = np.linalg.norm(out["out"] - ref["out"]) / np.linalg.norm(ref["out"])
    # E4M3 keeps 3 mantissa bits: rounding error uniform within half a step is ~2.6 % rms per operand, ~3.7 % per
    # product and (random signs) per dot product, ~5.5 % after silu(g) * u, ~6.6 % after the second quantised GEMM
    assert 3e-2 < rel < 1e-1, rel


def _read_fp8_golden():
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "fp8_hand_example.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if "=" in line:
                name, rhs = line.split("=")
                vals[name.strip()] = [int(v, 16) if v.lower().startswith("0x") else float(v) for v in rhs.split()]
    return vals


def test_hand_derived_fp8_example():
    """tests/golden/fp8_hand_example.txt: rows quantised by hand (exact codes, a rounding case, both tie cases, the
    all-zero row) and one expert followed through GEMM1, SwiGLU, the bf16 store, the re-quantisation and GEMM2."""
    g = _read_fp8_golden()
    rows = np.array(g["rows"], np.float32).reshape(4, 4)
    bits = _bf16_bits(rows)
    assert np.array_equal(oracle.bf16_to_f32(bits), rows)  # the example's inputs are bf16 values
    q, s = oracle.quantize_rows(bits)
    assert [int(c) for c in q.reshape(-1)] == g["codes"]
    assert np.array_equal(s, np.array(g["scales"], np.float64).astype(np.float32))
    wq1 = np.array(g["gate_up_codes"], np.uint8).reshape(2, 4)
    sw1 = np.array(g["gate_up_scale"], np.float32)
    act = oracle.gemm1_fp8(q[:1], s[:1], wq1, sw1)
    assert [int(v) for v in act.reshape(-1)] == g["act_bf16"]
    aq, sa = oracle.quantize_rows(act)
    assert int(aq[0, 0]) == 0xFE and sa[0] == np.float32(0.453125) / np.float32(448.0)
    wq2 = np.array(g["down_codes"], np.uint8).reshape(4, 1)
    sw2 = np.array(g["down_scale"], np.float32)
    y = oracle.gemm2_fp8(aq, sa, wq2, sw2)
    assert np.allclose(y[0], np.array(g["y"], np.float64), rtol=1e-6, atol=0)
    y_all = oracle.ffn_fp8(bits[:1], wq1, sw1, wq2, sw2)
    assert np.array_equal(y_all, y)
