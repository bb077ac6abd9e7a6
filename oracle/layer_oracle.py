"""CPU oracle for one decoder layer with multi-LoRA projections (TEST INFRASTRUCTURE ONLY).

Section 3.2 saves, per fine-tuning token, only the residual-stream input of each transformer layer
and lets the backward recompute the layer from it; Section 5 puts the adapters on the projection
matrices of a Llama-3-style layer.  This file states that layer in plain PyTorch CPU ops, float64,
with autograd doing the chain rule:

    h1 = RMSNorm(x; g1);   q, k, v = LoRA-projections(h1);   rotary embedding on q, k per sequence
    a  = causal softmax attention inside each sequence (grouped-query: kv heads shared by n_heads / n_kv heads)
    x2 = x + LoRA-projection_o(a);   h2 = RMSNorm(x2; g2)
    y  = x2 + LoRA-projection_down( SiLU(LoRA-projection_gate(h2)) * LoRA-projection_up(h2) )

A LoRA projection maps row t to  x_t W + s_a (x_t A_a^T) B_a  with the row's adapter a (none: base only).
Sequences are the segments of the table (a decode row is a one-token sequence here: no KV cache).
Readings: RMSNorm with eps 1e-5 and a learned gain, rotary base 500000 with the rotate-half pairing,
no biases - the Llama-3 conventions; the paper names the model, not these details.

Pins (tests/test_layer_pins.py): RMSNorm and rotary embedding against hand-computed values and their
defining properties (unit RMS; norm preservation and dependence on relative position only), causality
and independence of sequences, B = 0 gives the base layer, central finite differences for the
adapter and input gradients, and the wiring written out as literals: the SiLU gate against a hand value
that tells gate from up, both residual connections (all projections zero returns the input; the attention
branch alone gives 2 x), the 1 / sqrt(d_head) softmax scale on a two-token example with weights (1/4, 3/4),
the grouped-query head mapping on constant key-value heads, and lora_linear against the hot path's own
oracle (mlora_oracle.forward) on a mixed table.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence

import numpy as np
import torch

PROJ = ("q", "k", "v", "o", "gate", "up", "down")


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float = 1e-5) -> torch.Tensor:
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps) * gain


def rope(x: torch.Tensor, positions: torch.Tensor, theta: float = 500000.0) -> torch.Tensor:
    """x [T, heads, d_head]; pairs (i, i + d_head/2) are rotated by positions * theta^(-2i/d_head)."""
    d = x.shape[-1]
    half = d // 2
    inv = theta ** (-torch.arange(0, half, dtype=x.dtype) * 2.0 / d)
    ang = positions.to(x.dtype)[:, None] * inv[None, :]
    cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def lora_linear(x, W, A_all, B_all, scale, row_adapter) -> torch.Tensor:
    y = x @ W
    for a in sorted(set(int(v) for v in row_adapter if v >= 0)):
        rows = torch.tensor([t for t, v in enumerate(row_adapter) if v == a], dtype=torch.long)
        y = y.index_add(0, rows, scale[a] * ((x[rows] @ A_all[a].T) @ B_all[a]))
    return y


def attention(q, k, v, sequences: Sequence[Sequence[int]]) -> torch.Tensor:
    """q [T, H, dh], k, v [T, Hkv, dh]; causal softmax attention inside each sequence (list of rows in order)."""
    T, H, dh = q.shape
    rep = H // k.shape[1]
    out = torch.zeros_like(q)
    for rows in sequences:
        idx = torch.tensor(list(rows), dtype=torch.long)
        qs, ks, vs = q[idx], k[idx].repeat_interleave(rep, dim=1), v[idx].repeat_interleave(rep, dim=1)
        n = len(rows)
        s = torch.einsum("ihd,jhd->hij", qs, ks) / math.sqrt(dh)
        mask = torch.triu(torch.ones(n, n, dtype=torch.bool), diagonal=1)
        s = s.masked_fill(mask[None], float("-inf"))
        p = torch.softmax(s, dim=-1)
        out = out.index_copy(0, idx, torch.einsum("hij,jhd->ihd", p, vs))
    return out


def layer_forward(x, params: Dict, row_adapter, sequences, n_heads: int, n_kv: int) -> torch.Tensor:
    """params: g1, g2 [d]; for each projection name p: W_p, A_p, B_p, s_p."""
    T, d = x.shape
    dh = d // n_heads
    pos = torch.zeros(T, dtype=torch.long)
    for rows in sequences:
        for i, t in enumerate(rows):
            pos[t] = i
    lin = lambda name, inp: lora_linear(inp, params["W_" + name], params["A_" + name], params["B_" + name],
                                        params["s_" + name], row_adapter)
    h1 = rmsnorm(x, params["g1"])
    q = rope(lin("q", h1).reshape(T, n_heads, dh), pos)
    k = rope(lin("k", h1).reshape(T, n_kv, dh), pos)
    v = lin("v", h1).reshape(T, n_kv, dh)
    a = attention(q, k, v, sequences).reshape(T, d)
    x2 = x + lin("o", a)
    h2 = rmsnorm(x2, params["g2"])
    m = torch.nn.functional.silu(lin("gate", h2)) * lin("up", h2)
    return x2 + lin("down", m)


def layer_backward(x, params: Dict, row_adapter, sequences, n_heads: int, n_kv: int, dy, adapters: Sequence[int]):
    """Recompute the layer from its input (the only saved state) and return dx and, for each projection,
    dA [len(adapters), r, d_in] and dB [len(adapters), r, d_out] of the listed adapters."""
    x = x.clone().requires_grad_(True)
    p = {k: (v.clone().requires_grad_(True) if k[:2] in ("A_", "B_") else v) for k, v in params.items()}
    y = layer_forward(x, p, row_adapter, sequences, n_heads, n_kv)
    y.backward(dy)
    out = {"dx": x.grad.detach()}
    for name in PROJ:
        out["dA_" + name] = torch.stack([p["A_" + name].grad[a] for a in adapters]).detach()
        out["dB_" + name] = torch.stack([p["B_" + name].grad[a] for a in adapters]).detach()
    return out
