"""One decoder layer chained through the library's projections, with the paper's default activation
policy (Section 3.2): the serving forward keeps only the layer's residual-stream input for the
fine-tuning rows; the backward recomputes the layer from it, over the fine-tuning rows alone, and
returns the LoRA gradients of all seven projections and the gradient of the layer input (what the
layer below needs).

Division of labour: every arithmetic step of the layer is a kernel of this library - the seven projections
(q, k, v, o, gate, up, down) through `mlora_mixed_forward` (serving pass, recompute pass) and
`mlora_backward`; RMSNorm, the rotary embedding, the SiLU gate, the residual adds and attention with
their input gradients through the entry points of `mlora_layer_ops.h` (attention on the tcgen05 kernels
for head size 128, CUDA-core kernels for head size 64).  The backward is written out call by call: where
a tensor feeds several consumers (the layer input feeds the norm and the residual, the normed input feeds
q, k and v, the second normed input feeds gate and up) the gradients are summed by `mlora_add`.  PyTorch
only owns the buffers.  A decode row is a one-token sequence (no KV cache in this module).
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

    # -- layer body; `lin(name, x)` is the projection call; returns the output and every intermediate ---
    def _body(self, x, lin, sequences, tables=None):
        T = x.shape[0]
        dh = self.d // self.n_heads
        dev = x.device
        pos, seq_start, seq_end = tables if tables is not None else (torch.from_numpy(t).to(dev) for t in sequence_tables(T, sequences))
        new = torch.empty_like
        t = {"x": x, "pos": pos, "seq_start": seq_start, "seq_end": seq_end}
        t["h1"] = new(x); mo.mlora_rmsnorm_forward(x, self.g1, t["h1"])
        q0, k0, t["v"] = lin("q", t["h1"]), lin("k", t["h1"]), lin("v", t["h1"])
        t["q"], t["k"] = new(q0), new(k0)
        mo.mlora_rope(q0, t["q"], pos, self.n_heads, dh)
        mo.mlora_rope(k0, t["k"], pos, self.n_kv, dh)
        t["a"] = new(t["q"])
        t["lse"] = torch.empty((T, self.n_heads), dtype=torch.float32, device=dev)
        mo.mlora_attention_forward(t["q"], t["k"], t["v"], t["a"], t["lse"], seq_start, seq_end, self.n_heads, self.n_kv, dh)
        t["x2"] = new(x); mo.mlora_add(x, lin("o", t["a"]), t["x2"])
        t["h2"] = new(x); mo.mlora_rmsnorm_forward(t["x2"], self.g2, t["h2"])
        t["g"], t["u"] = lin("gate", t["h2"]), lin("up", t["h2"])
        t["m"] = new(t["g"]); mo.mlora_swiglu_forward(t["g"], t["u"], t["m"])
        y = new(x); mo.mlora_add(t["x2"], lin("down", t["m"]), y)
        return y, t

    # -- serving forward: mixed batch, keeps the layer input of the fine-tuning rows --------------
    @torch.no_grad()
    def forward(self, x, segments: np.ndarray) -> torch.Tensor:
        """segments cover the batch contiguously in row order (every segment is one sequence)."""
        segs = np.asarray(segments, dtype=np.int32).reshape(-1, 4)
        n_rows = x.shape[0]
        serving = segs.copy()
        serving[:, 3] = 0                           # projection-level saves are not kept: the policy saves the layer input
        # a plan per batch, from the context's pool and ordered on the stream: no allocation, no synchronisation
        plan = mb.mlora_plan_create_async(self.sess.ctx, serving, n_rows, self.n_adapters)
        try:
            def lin(name, inp):
                pr = self.proj[name]
                y = torch.empty((n_rows, pr.d_out), dtype=torch.bfloat16, device=x.device)
                mb.mlora_mixed_forward(self.sess.ctx, pr.layer, plan, inp.contiguous(), y, None, None, 0, 0)
                return y
            y, _ = self._body(x, lin, segs[segs[:, 1] > 0][:, :2])
        finally:
            mb.mlora_plan_release(plan)
        # activation capture: the residual-stream input of the fine-tuning rows
        for s, n, a, _ in segs[(segs[:, 3] != 0) & (segs[:, 1] > 0)]:
            self.saved_x[self.saved_rows:self.saved_rows + n] = x[s:s + n]
            self.saved.append((int(n), int(a)))
            self.saved_rows += int(n)
        return y

    # -- the serving forward of one batch shape as a CUDA graph ------------------------------------
    @torch.no_grad()
    def capture_forward(self, x, segments: np.ndarray):
        """The serving forward (no activation capture) of this batch layout captured once and replayed: the ~30
        launches of the layer leave the host as one graph launch.  Every call of the library is allocation-free
        and never synchronises, which is what makes the capture possible; the plan and the sequence tables are
        made before it.  Returns an object with ``x`` (static input buffer: copy the batch into it), ``y`` (static
        output), ``replay()`` and ``close()``."""
        segs = np.asarray(segments, dtype=np.int32).reshape(-1, 4)
        n_rows = x.shape[0]
        serving = segs.copy()
        serving[:, 3] = 0
        plan = mb.mlora_plan_create(self.sess.ctx, serving, n_rows, self.n_adapters)
        dev = x.device
        tables = tuple(torch.from_numpy(t).to(dev) for t in sequence_tables(n_rows, segs[segs[:, 1] > 0][:, :2]))
        layer = self

        def lin(name, inp):
            pr = layer.proj[name]
            y = torch.empty((n_rows, pr.d_out), dtype=torch.bfloat16, device=dev)
            mb.mlora_mixed_forward(layer.sess.ctx, pr.layer, plan, inp, y, None, None, 0, 0)
            return y

        class Captured:
            pass
        cap = Captured()
        cap.tables = tables                      # the graph's kernels read them on every replay
        cap.x = x.clone()
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for _ in range(2):                   # one-time function attributes and per-plan lists are made here
                self._body(cap.x, lin, None, tables)
            stream.synchronize()
            cap.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cap.graph, stream=stream):
                cap.y, _ = self._body(cap.x, lin, None, tables)
        cap.replay = cap.graph.replay

        def close():
            torch.cuda.synchronize()
            mb.mlora_plan_destroy(plan)
        cap.close = close
        return cap

    # -- backward: recompute from the saved layer input, fine-tuning rows only ---------------------
    def _backward_body(self, x, dy, plan, n_slots, sequences, tables=None):
        """Recompute the layer over the saved rows `x` and backpropagate `dy`; every call is a library kernel."""
        rows = x.shape[0]
        dev, ctx = x.device, self.sess.ctx
        dh = self.d // self.n_heads

        def lin(name, inp):          # recompute pass: every row is a fine-tuning row, each projection saves its own input and x A^T
            pr = self.proj[name]
            y = torch.empty((rows, pr.d_out), dtype=torch.bfloat16, device=dev)
            mb.mlora_mixed_forward(ctx, pr.layer, plan, inp, y, pr.x_save, pr.u_save, 0, pr.x_save.shape[0])
            return y

        def lin_bwd(name, g):        # LoRA gradients of one projection and the gradient of its input
            pr = self.proj[name]
            pr.dA = torch.empty((n_slots, pr.rank, pr.d_in), dtype=torch.float32, device=dev)
            pr.dB = torch.empty((n_slots, pr.rank, pr.d_out), dtype=torch.float32, device=dev)
            dx = torch.empty((rows, pr.d_in), dtype=torch.bfloat16, device=dev)
            mb.mlora_backward(ctx, pr.layer, plan, g, pr.x_save, pr.u_save, pr.dA, pr.dB, dx)
            return dx

        _y, t = self._body(x, lin, sequences, tables)
        # y = x2 + down(m): dy reaches x2 directly and through the feed-forward branch
        dm = lin_bwd("down", dy)
        dg, du = torch.empty_like(t["g"]), torch.empty_like(t["u"])
        mo.mlora_swiglu_backward(t["g"], t["u"], dm, dg, du)
        dh2 = lin_bwd("gate", dg)
        mo.mlora_add(dh2, lin_bwd("up", du), dh2)                   # h2 feeds gate and up
        dx2 = torch.empty_like(x)
        mo.mlora_rmsnorm_backward(t["x2"], self.g2, dh2, dx2)
        mo.mlora_add(dx2, dy, dx2)                                  # x2 feeds the norm and the residual
        # x2 = x + o(a)
        da = lin_bwd("o", dx2)
        dq, dk, dv = torch.empty_like(t["q"]), torch.empty_like(t["k"]), torch.empty_like(t["v"])
        mo.mlora_attention_backward(t["q"], t["k"], t["v"], t["a"], t["lse"], da, dq, dk, dv, t["seq_start"], t["seq_end"],
                                    self.n_heads, self.n_kv, dh)
        dq0, dk0 = torch.empty_like(dq), torch.empty_like(dk)
        mo.mlora_rope(dq, dq0, t["pos"], self.n_heads, dh, transpose=True)
        mo.mlora_rope(dk, dk0, t["pos"], self.n_kv, dh, transpose=True)
        dh1 = lin_bwd("q", dq0)
        mo.mlora_add(dh1, lin_bwd("k", dk0), dh1)                   # h1 feeds q, k and v
        mo.mlora_add(dh1, lin_bwd("v", dv), dh1)
        dx = torch.empty_like(x)
        mo.mlora_rmsnorm_backward(x, self.g1, dh1, dx)
        mo.mlora_add(dx, dx2, dx)                                   # x feeds the norm and the residual
        grads = {n: (self.proj[n].dA, self.proj[n].dB) for n in PROJ}
        return dx, grads

    @staticmethod
    def _saved_table(saved):
        table, row = [], 0
        for n, a in saved:
            table.append((row, n, a, 1)); row += n
        return synth.segments_array(table), row

    def backward(self, dy_ft: torch.Tensor):
        """dy_ft [saved rows, d]: gradient of the layer output for the saved rows, in save order.
        Returns (dx [saved rows, d], {projection: (dA, dB)}, adapters of the gradient slots)."""
        rows = self.saved_rows
        table, _ = self._saved_table(self.saved)
        self.bwd_plan = mb.mlora_plan_create_async(self.sess.ctx, table, rows, self.n_adapters)
        self.bwd_slots = mb.mlora_plan_ft_adapters(self.bwd_plan)
        try:
            x = self.saved_x[:rows]
            dy = dy_ft.to(torch.bfloat16).contiguous()
            dx, grads = self._backward_body(x, dy, self.bwd_plan, len(self.bwd_slots), [(int(s), int(n)) for s, n, _, _ in table])
            torch.cuda.synchronize()
            return dx, grads, list(self.bwd_slots)
        finally:
            mb.mlora_plan_release(self.bwd_plan)
            self.bwd_plan = None
            self.saved, self.saved_rows = [], 0

    @torch.no_grad()
    def capture_backward(self, saved):
        """The recompute + backward over a fixed layout of saved fine-tuning sequences (`saved`: (tokens, adapter) in
        save order, e.g. the paper's backward batches of 256 tokens) captured once in a CUDA graph.  The layer input
        of those rows is read from the layer's own save buffer (where the serving forwards put it), `dy` is a static
        buffer to copy the output gradient into.  Returns an object with ``dy``, ``dx``, ``grads`` (static outputs),
        ``slots``, ``replay()`` and ``close()``."""
        table, rows = self._saved_table(saved)
        plan = mb.mlora_plan_create(self.sess.ctx, table, rows, self.n_adapters)
        slots = mb.mlora_plan_ft_adapters(plan)
        dev = self.saved_x.device
        seqs = [(int(s), int(n)) for s, n, _, _ in table]
        tables = tuple(torch.from_numpy(t).to(dev) for t in sequence_tables(rows, seqs))
        x = self.saved_x[:rows]

        class Captured:
            pass
        cap = Captured()
        cap.tables = tables                      # the graph's kernels read them on every replay
        cap.dy = torch.zeros((rows, self.d), dtype=torch.bfloat16, device=dev)
        cap.slots = list(slots)
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for _ in range(2):
                self._backward_body(x, cap.dy, plan, len(slots), None, tables)
            stream.synchronize()
            cap.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cap.graph, stream=stream):
                cap.dx, cap.grads = self._backward_body(x, cap.dy, plan, len(slots), None, tables)
        cap.replay = cap.graph.replay

        def close():
            torch.cuda.synchronize()
            mb.mlora_plan_destroy(plan)
        cap.close = close
        return cap
