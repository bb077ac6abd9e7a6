"""One decoder layer chained through the library's projections, with the paper's default activation
policy (Section 3.2): the serving forward keeps only the layer's residual-stream input for the
fine-tuning rows; the backward recomputes the layer from it, over the fine-tuning rows alone, and
returns the LoRA gradients of all seven projections and the gradient of the layer input (what the
layer below needs).

Division of labour: the seven projections (q, k, v, o, gate, up, down) run in this library's kernels
- `mlora_mixed_forward` in the serving pass, `mlora_mixed_forward` + `mlora_backward` in the
recompute/backward pass - and so do RMSNorm, the rotary embedding, the SiLU gate and the residual adds
with their input gradients, and attention as a plain CUDA-core kernel pair for short sequences
(`mlora_layer_ops.h`).  PyTorch's autograd only strings the pieces together; every arithmetic step of
the layer runs in this library.  A decode row is a one-token sequence (no KV cache in this module).
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

from . import binding as mb
from . import layer_ops as mo
from . import synth

PROJ = ("q", "k", "v", "o", "gate", "up", "down")


class _Projection:
    def __init__(self, sess, W, A_all, B_all, scale, cap_rows):
        dev = sess.device
        self.W, self.A, self.B = (t.to(dev).to(torch.bfloat16).contiguous() for t in (W, A_all, B_all))
        self.scale = scale.to(dev).to(torch.float32).contiguous()
        self.layer = mb.make_layer(self.W, self.A, self.B, self.scale)
        self.d_in, self.d_out, self.rank = self.W.shape[0], self.W.shape[1], self.A.shape[1]
        self.x_save = torch.empty((cap_rows, self.d_in), dtype=torch.bfloat16, device=dev)
        self.u_save = torch.empty((cap_rows, self.rank), dtype=torch.float32, device=dev)
        self.dA = self.dB = None


class _ProjFn(torch.autograd.Function):
    """A multi-LoRA projection over a batch whose rows are all fine-tuning rows (the recompute pass)."""

    @staticmethod
    def forward(ctx, x, owner, name):
        pr = owner.proj[name]
        x = x.contiguous()
        y = torch.empty((x.shape[0], pr.d_out), dtype=torch.bfloat16, device=x.device)
        mb.mlora_mixed_forward(owner.sess.ctx, pr.layer, owner.bwd_plan, x, y, pr.x_save, pr.u_save, 0, pr.x_save.shape[0])
        ctx.owner, ctx.name = owner, name
        return y

    @staticmethod
    def backward(ctx, dy):
        owner, pr = ctx.owner, ctx.owner.proj[ctx.name]
        dy = dy.to(torch.bfloat16).contiguous()
        n_slots = len(owner.bwd_slots)
        pr.dA = torch.empty((n_slots, pr.rank, pr.d_in), dtype=torch.float32, device=dy.device)
        pr.dB = torch.empty((n_slots, pr.rank, pr.d_out), dtype=torch.float32, device=dy.device)
        dx = torch.empty((dy.shape[0], pr.d_in), dtype=torch.bfloat16, device=dy.device)
        mb.mlora_backward(owner.sess.ctx, pr.layer, owner.bwd_plan, dy, pr.x_save, pr.u_save, pr.dA, pr.dB, dx)
        return dx, None, None


class _RmsNormFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, gain):
        x = x.contiguous()
        y = torch.empty_like(x)
        mo.mlora_rmsnorm_forward(x, gain, y)
        ctx.save_for_backward(x, gain)
        return y

    @staticmethod
    def backward(ctx, dy):
        x, gain = ctx.saved_tensors
        dx = torch.empty_like(x)
        mo.mlora_rmsnorm_backward(x, gain, dy.contiguous(), dx)
        return dx, None


class _RopeFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, pos, n_heads, d_head):
        x = x.contiguous()
        y = torch.empty_like(x)
        mo.mlora_rope(x, y, pos, n_heads, d_head)
        ctx.pos, ctx.shape = pos, (n_heads, d_head)
        return y

    @staticmethod
    def backward(ctx, dy):
        dx = torch.empty_like(dy)
        mo.mlora_rope(dy.contiguous(), dx, ctx.pos, ctx.shape[0], ctx.shape[1], transpose=True)
        return dx, None, None, None


class _SwigluFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, g, u):
        g, u = g.contiguous(), u.contiguous()
        m = torch.empty_like(g)
        mo.mlora_swiglu_forward(g, u, m)
        ctx.save_for_backward(g, u)
        return m

    @staticmethod
    def backward(ctx, dm):
        g, u = ctx.saved_tensors
        dg, du = torch.empty_like(g), torch.empty_like(u)
        mo.mlora_swiglu_backward(g, u, dm.contiguous(), dg, du)
        return dg, du


class _AttnFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, seq_start, seq_end, n_heads, n_kv, d_head):
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        o = torch.empty_like(q)
        lse = torch.empty((q.shape[0], n_heads), dtype=torch.float32, device=q.device)
        mo.mlora_attention_forward(q, k, v, o, lse, seq_start, seq_end, n_heads, n_kv, d_head)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.meta = (seq_start, seq_end, n_heads, n_kv, d_head)
        return o

    @staticmethod
    def backward(ctx, dO):
        q, k, v, o, lse = ctx.saved_tensors
        seq_start, seq_end, n_heads, n_kv, d_head = ctx.meta
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        mo.mlora_attention_backward(q, k, v, o, lse, dO.contiguous(), dq, dk, dv, seq_start, seq_end, n_heads, n_kv, d_head)
        return dq, dk, dv, None, None, None, None, None


class _AddFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, a, b):
        out = torch.empty_like(a)
        mo.mlora_add(a.contiguous(), b.contiguous(), out)
        return out

    @staticmethod
    def backward(ctx, d):
        return d, d


def sequence_tables(n_rows: int, sequences) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Per-row position inside its sequence, first row and one-past-last row of its sequence (int32 [n_rows])
    for sequences given as (first row, length) pairs; rows outside every sequence stand alone.  Built on the
    host without a Python loop over the sequences."""
    start = np.arange(n_rows, dtype=np.int32)
    end = start + 1
    sq = np.asarray(sequences, dtype=np.int64).reshape(-1, 2)
    sq = sq[sq[:, 1] > 0]
    if len(sq):
        first = np.repeat(sq[:, 0], sq[:, 1])
        rows = first + (np.arange(int(sq[:, 1].sum())) - np.repeat(np.cumsum(sq[:, 1]) - sq[:, 1], sq[:, 1]))
        start[rows] = first
        end[rows] = np.repeat(sq[:, 0] + sq[:, 1], sq[:, 1])
    pos = (np.arange(n_rows, dtype=np.int32) - start).astype(np.int32)
    return pos, start, end


class DecoderLayer:
    def __init__(self, sess, params: Dict[str, torch.Tensor], n_heads: int, n_kv: int, max_ft_rows: int):
        """params as in the layer oracle: g1, g2, and W_p / A_p / B_p / s_p for the seven projections."""
        self.sess, self.n_heads, self.n_kv = sess, n_heads, n_kv
        dev = sess.device
        self.g1, self.g2 = params["g1"].to(dev).float(), params["g2"].to(dev).float()
        self.proj = {n: _Projection(sess, params["W_" + n], params["A_" + n], params["B_" + n], params["s_" + n], max_ft_rows)
                     for n in PROJ}
        self.n_adapters = params["A_q"].shape[0]
        self.d = params["W_q"].shape[0]
        self.saved_x = torch.empty((max_ft_rows, self.d), dtype=torch.bfloat16, device=dev)   # the layer-input buffer
        self.saved: List[Tuple[int, int]] = []      # (tokens, adapter) of the saved fine-tuning sequences, in save order
        self.saved_rows = 0
        self.bwd_plan, self.bwd_slots = None, []

    # -- shared layer body; `lin(name, x)` is the projection call ---------------------------------
    def _body(self, x, lin, sequences):
        T = x.shape[0]
        dh = self.d // self.n_heads
        pos, seq_start, seq_end = (torch.from_numpy(t).to(x.device) for t in sequence_tables(T, sequences))
        h1 = _RmsNormFn.apply(x, self.g1)
        q = _RopeFn.apply(lin("q", h1), pos, self.n_heads, dh)
        k = _RopeFn.apply(lin("k", h1), pos, self.n_kv, dh)
        v = lin("v", h1)
        a = _AttnFn.apply(q, k, v, seq_start, seq_end, self.n_heads, self.n_kv, dh)
        x2 = _AddFn.apply(x, lin("o", a))
        h2 = _RmsNormFn.apply(x2, self.g2)
        m = _SwigluFn.apply(lin("gate", h2), lin("up", h2))
        return _AddFn.apply(x2, lin("down", m))

    # -- serving forward: mixed batch, keeps the layer input of the fine-tuning rows --------------
    @torch.no_grad()
    def forward(self, x, segments: np.ndarray) -> torch.Tensor:
        """segments cover the batch contiguously in row order (every segment is one sequence)."""
        segs = np.asarray(segments, dtype=np.int32).reshape(-1, 4)
        n_rows = x.shape[0]
        serving = segs.copy()
        serving[:, 3] = 0                           # projection-level saves are not kept: the policy saves the layer input
        plan = mb.mlora_plan_create(self.sess.ctx, serving, n_rows, self.n_adapters)
        try:
            def lin(name, inp):
                pr = self.proj[name]
                y = torch.empty((n_rows, pr.d_out), dtype=torch.bfloat16, device=x.device)
                mb.mlora_mixed_forward(self.sess.ctx, pr.layer, plan, inp.contiguous(), y, None, None, 0, 0)
                return y
            y = self._body(x, lin, segs[segs[:, 1] > 0][:, :2])
        finally:
            torch.cuda.synchronize()
            mb.mlora_plan_destroy(plan)
        # activation capture: the residual-stream input of the fine-tuning rows
        for s, n, a, _ in segs[(segs[:, 3] != 0) & (segs[:, 1] > 0)]:
            self.saved_x[self.saved_rows:self.saved_rows + n] = x[s:s + n]
            self.saved.append((int(n), int(a)))
            self.saved_rows += int(n)
        return y

    # -- backward: recompute from the saved layer input, fine-tuning rows only ---------------------
    def backward(self, dy_ft: torch.Tensor):
        """dy_ft [saved rows, d]: gradient of the layer output for the saved rows, in save order.
        Returns (dx [saved rows, d], {projection: (dA, dB)}, adapters of the gradient slots)."""
        rows = self.saved_rows
        table, row = [], 0
        for n, a in self.saved:
            table.append((row, n, a, 1)); row += n
        table = synth.segments_array(table)
        self.bwd_plan = mb.mlora_plan_create(self.sess.ctx, table, rows, self.n_adapters)
        self.bwd_slots = mb.mlora_plan_ft_adapters(self.bwd_plan)
        try:
            x = self.saved_x[:rows].clone().requires_grad_(True)
            with torch.enable_grad():
                y = self._body(x, lambda name, inp: _ProjFn.apply(inp, self, name), [(int(s), int(n)) for s, n, _, _ in table])
                y.backward(dy_ft.to(torch.bfloat16))
            torch.cuda.synchronize()
            grads = {n: (self.proj[n].dA, self.proj[n].dB) for n in PROJ}
            return x.grad, grads, list(self.bwd_slots)
        finally:
            mb.mlora_plan_destroy(self.bwd_plan)
            self.bwd_plan = None
            self.saved, self.saved_rows = [], 0
