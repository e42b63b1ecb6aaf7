"""Seeded synthetic inputs for the MoE layer -- shapes and value distributions only.

This module is the one thing the CUDA path's tests and the CPU oracle's tests
both use.  It holds none of the layer's arithmetic: it draws activations,
router logits, selection bias and weights with the distributions the five
workloads specify, and nothing else.  It imports torch only.

Workloads (the paper's evaluation prints only model shapes -- top-8 routing
over hundreds of experts, bf16 -- and trace statistics: prefill increments of
hundreds to a few thousand tokens, decode batches of at most ~128 sequences;
the five shapes below stand in for its internal checkpoints and trace):

  C1  tiny prefill        T=64    H=256   E=8    k=2  I=512   no shared expert
  C2  decode, V3-shaped   T=128   H=7168  E=256  k=8  I=2048  + shared expert (I=2048), selection bias
  C3  prefill, Qwen3-30B  T=8192  H=2048  E=128  k=8  I=768   no shared expert, chunked prompt lengths
  C4  P/D multiplexing    C2's layer; P batch T=4096 and D batch T=64 on two streams
  C5  skewed sweep        C2's layer; logits = N(0,1) + log Zipf(1.2) weight; T in {1,...,32768}
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch


@dataclasses.dataclass(frozen=True)
class LayerShape:
    name: str
    T: int            # tokens per call
    H: int            # hidden size
    E: int            # routed experts
    k: int            # experts per token
    I: int            # routed expert intermediate size
    shared_I: int = 0  # shared expert intermediate size (0 = no shared expert)
    select_bias: bool = False
    zipf_s: float = 0.0  # >0: add log Zipf(s) popularity to the logits

    @property
    def N(self) -> int:
        return self.T * self.k

    def with_tokens(self, T: int) -> "LayerShape":
        return dataclasses.replace(self, T=T)


C1 = LayerShape("C1-tiny", T=64, H=256, E=8, k=2, I=512)
C2 = LayerShape("C2-decode-v3", T=128, H=7168, E=256, k=8, I=2048, shared_I=2048, select_bias=True)
C3 = LayerShape("C3-prefill-qwen3", T=8192, H=2048, E=128, k=8, I=768)
C4_P = LayerShape("C4-P-v3", T=4096, H=7168, E=256, k=8, I=2048, shared_I=2048, select_bias=True)
C4_D = LayerShape("C4-D-v3", T=64, H=7168, E=256, k=8, I=2048, shared_I=2048, select_bias=True)
C5 = LayerShape("C5-zipf-v3", T=1024, H=7168, E=256, k=8, I=2048, shared_I=2048, zipf_s=1.2)
C5_TOKENS = (1, 16, 128, 1024, 8192, 32768)

WORKLOADS = {"C1": C1, "C2": C2, "C3": C3, "C4P": C4_P, "C4D": C4_D, "C5": C5}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_weights(shape: LayerShape, seed: int, device="cpu") -> dict:
    """Random-init layer weights ~ N(0, 0.02) in bf16.

    w_gate_up [E, 2I, H] (rows 0..I-1 gate, I..2I-1 up), w_down [E, H, I];
    ws_gate_up [2Is, H], ws_down [H, Is] when the shape has a shared expert.
    Drawn one expert at a time so that the fp32 staging stays small.
    """
    g = _gen(seed, device)
    w_gate_up = torch.empty(shape.E, 2 * shape.I, shape.H, dtype=torch.bfloat16, device=device)
    w_down = torch.empty(shape.E, shape.H, shape.I, dtype=torch.bfloat16, device=device)
    for e in range(shape.E):
        w_gate_up[e].copy_(torch.randn(2 * shape.I, shape.H, generator=g, device=device) * 0.02)
        w_down[e].copy_(torch.randn(shape.H, shape.I, generator=g, device=device) * 0.02)
    out = {"w_gate_up": w_gate_up, "w_down": w_down, "ws_gate_up": None, "ws_down": None}
    if shape.shared_I:
        out["ws_gate_up"] = (torch.randn(2 * shape.shared_I, shape.H, generator=g, device=device) * 0.02).to(torch.bfloat16)
        out["ws_down"] = (torch.randn(shape.H, shape.shared_I, generator=g, device=device) * 0.02).to(torch.bfloat16)
    return out


def make_weights_fp8(shape: LayerShape, seed: int, device="cpu", std: float = 0.02) -> dict:
    """Random-init layer weights in the FP8 checkpoint format: E4M3 codes (uint8) plus one fp32 scale per output
    channel.  A channel's codes are N(0, 112) clamped to the E4M3 range and converted by torch's own float8 type
    (4 sigma reaches the largest code, as a per-channel absmax quantiser would produce); its scale is
    std / 112 times a factor drawn from [0.8, 1.2], so that scale * code ~ N(0, std) like the bf16 weights.

    wq_gate_up [E, 2I, H], sw_gate_up [E, 2I], wq_down [E, H, I], sw_down [E, H]; with a shared expert also
    wsq_gate_up [2Is, H], sws_gate_up [2Is], wsq_down [H, Is], sws_down [H].
    """
    g = _gen(seed, device)

    def codes(rows, cols):
        v = (torch.randn(rows, cols, generator=g, device=device) * 112.0).clamp_(-448.0, 448.0)
        return v.to(torch.float8_e4m3fn).view(torch.uint8)

    def scales(*dims):
        return ((0.8 + 0.4 * torch.rand(*dims, generator=g, device=device)) * (std / 112.0)).float()

    wq_gate_up = torch.empty(shape.E, 2 * shape.I, shape.H, dtype=torch.uint8, device=device)
    wq_down = torch.empty(shape.E, shape.H, shape.I, dtype=torch.uint8, device=device)
    for e in range(shape.E):
        wq_gate_up[e].copy_(codes(2 * shape.I, shape.H))
        wq_down[e].copy_(codes(shape.H, shape.I))
    out = {"wq_gate_up": wq_gate_up, "sw_gate_up": scales(shape.E, 2 * shape.I), "wq_down": wq_down,
           "sw_down": scales(shape.E, shape.H), "wsq_gate_up": None, "sws_gate_up": None, "wsq_down": None,
           "sws_down": None}
    if shape.shared_I:
        out["wsq_gate_up"] = codes(2 * shape.shared_I, shape.H)
        out["sws_gate_up"] = scales(2 * shape.shared_I)
        out["wsq_down"] = codes(shape.H, shape.shared_I)
        out["sws_down"] = scales(shape.H)
    return out


def zipf_log_weight(E: int, s: float, seed: int, device="cpu") -> torch.Tensor:
    """log of Zipf(s) popularity per expert id: rank r in 1..E gets r^-s, ranks
    assigned to expert ids by a seeded permutation (hot experts are not adjacent)."""
    g = _gen(seed, "cpu")
    ranks = torch.randperm(E, generator=g) + 1
    return (-s * torch.log(ranks.double())).float().to(device)


def make_activations(shape: LayerShape, seed: int, device="cpu", T: Optional[int] = None) -> dict:
    """Per-call inputs: x ~ N(0,1) bf16 [T,H]; router logits ~ N(0,1) fp32 [T,E]
    (+ log Zipf popularity when the shape asks for it); selection bias ~ N(0,0.5)
    fp32 [E] or None."""
    T = shape.T if T is None else T
    g = _gen(seed, device)
    x = torch.randn(T, shape.H, generator=g, device=device).to(torch.bfloat16)
    logits = torch.randn(T, shape.E, generator=g, device=device)
    bias = None
    if shape.select_bias:
        bias = torch.randn(shape.E, generator=g, device=device) * 0.5
    if shape.zipf_s > 0:
        logits = logits + zipf_log_weight(shape.E, shape.zipf_s, seed + 7919, device)[None, :]
    return {"x": x.contiguous(), "logits": logits.contiguous(), "bias": bias}


def prefill_chunk_lengths(total: int, seed: int, lo: int = 512, hi: int = 4096) -> list:
    """Prompt-chunk lengths U{lo..hi} concatenated (last one truncated) to `total` tokens."""
    g = _gen(seed, "cpu")
    out, acc = [], 0
    while acc < total:
        n = int(torch.randint(lo, hi + 1, (1,), generator=g).item())
        n = min(n, total - acc)
        out.append(n)
        acc += n
    return out


def tie_heavy_logits(T: int, E: int, seed: int, device="cpu") -> torch.Tensor:
    """Logits quantised to multiples of 0.25 with a mixture of +0.0 and -0.0, so
    that equal keys are common and the tie rule is exercised."""
    g = _gen(seed, device)
    q = torch.randint(-4, 5, (T, E), generator=g, device=device).float() * 0.25
    neg_zero = torch.rand(T, E, generator=g, device=device) < 0.5
    return torch.where((q == 0) & neg_zero, torch.full_like(q, -0.0), q).contiguous()


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
