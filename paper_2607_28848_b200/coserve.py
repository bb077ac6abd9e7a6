"""A single-process co-serving loop over one multi-LoRA projection: the paper's pipeline (Section 3.2,
Section 4.2) expressed with this library's entry points.

Per step the host proposes an inference batch; `mlora_sched_admit` (Algorithm 1, priced with Eq. I)
picks fine-tuning samples that fit the SLO budget and the activation buffer; the step's segment
table carries prefill requests, decode rows and the admitted samples; `mlora_mixed_forward` runs it
and appends the fine-tuning rows' activations behind those already saved.  When a step holds no
prefill tokens (the backward yields to prefill, Section 4.2 "Backward preemption") and at least
`backward_batch` tokens are saved, `mlora_backward` + `mlora_adamw_update` consume the saved rows
and the scheduler gets the buffer back.  An interrupted fine-tuning forward returns its samples to
the pool (`mlora_sched_requeue`).

The loop itself is host logic and runs against any executor with `forward / backward / update`;
`GpuExecutor` is the one that calls the CUDA library.  `python -m paper_2607_28848_b200.coserve`
runs a synthetic arrival pattern on one GPU and prints a summary table.
"""
from __future__ import annotations

import argparse
import sys
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import sched as ms
from . import synth


@dataclass
class SavedSample:
    sample_id: int
    tokens: int
    adapter: int


class CoServeLoop:
    def __init__(self, executor, scheduler, n_adapters: int, ft_adapter_of=lambda sample_id: 0,
                 backward_batch: int = 256):
        self.ex, self.s = executor, scheduler
        self.n_adapters = n_adapters
        self.ft_adapter_of = ft_adapter_of
        self.backward_batch = backward_batch
        self.saved: List[SavedSample] = []          # activation buffer contents, in save order
        self.saved_tokens = 0
        self.trained: List[int] = []                # sample ids whose backward has run
        self.n_backward = 0

    # -- segment tables ---------------------------------------------------------------------
    def _step_table(self, prefill: Sequence[Tuple[int, int]], decode_adapters: Sequence[int],
                    ft: Sequence[SavedSample]) -> Tuple[np.ndarray, int]:
        segs, row = [], 0
        for n, a in prefill:
            segs.append((row, n, a, 0)); row += n
        for a in decode_adapters:
            segs.append((row, 1, a, 0)); row += 1
        for smp in ft:
            segs.append((row, smp.tokens, smp.adapter, 1)); row += smp.tokens
        return synth.segments_array(segs), row

    def _backward_table(self) -> Tuple[np.ndarray, int]:
        segs, row = [], 0
        for smp in self.saved:                       # save order = row order of the compact table
            segs.append((row, smp.tokens, smp.adapter, 1)); row += smp.tokens
        return synth.segments_array(segs), row

    # -- one scheduling step ----------------------------------------------------------------
    def step(self, prefill: Sequence[Tuple[int, int]], decode_adapters: Sequence[int], kv_tokens: int, t_now: float,
             earliest_arrival: Optional[float], interrupt: bool = False) -> Dict:
        lens = [n for n, _ in prefill]
        ids, toks, budget = ms.mlora_sched_admit(self.s, lens, len(decode_adapters), kv_tokens, t_now,
                                                 earliest_arrival if lens else None)
        ft = [SavedSample(i, t, self.ft_adapter_of(i)) for i, t in zip(ids, toks)]
        table, n_rows = self._step_table(prefill, decode_adapters, ft)
        out = {"admitted": list(ids), "ft_tokens": int(sum(toks)), "rows": n_rows, "budget": budget,
               "backward": False, "interrupted": False}
        if n_rows:
            done = self.ex.forward(table, n_rows, self.saved_tokens, cancel=interrupt)
            if not done:                             # interrupted: partial activations are dropped by not
                ms.mlora_sched_requeue(self.s, ids, toks)   # advancing the save base; the samples return to the pool
                out.update(interrupted=True, admitted=[], ft_tokens=0)
                return out
        self.saved += ft
        self.saved_tokens += int(sum(toks))
        if not lens and self.saved_tokens >= self.backward_batch:
            ms.mlora_sched_set_backward_running(self.s, True)
            table_b, rows_b = self._backward_table()
            self.ex.backward(table_b, rows_b)
            self.ex.update(table_b, rows_b)
            ms.mlora_sched_buffer_release(self.s, self.saved_tokens)
            ms.mlora_sched_set_backward_running(self.s, False)
            self.trained += [smp.sample_id for smp in self.saved]
            self.saved, self.saved_tokens = [], 0
            self.n_backward += 1
            out["backward"] = True
        return out


class GpuExecutor:
    """Runs the loop's steps through the CUDA library on one projection (d_in -> d_out, bf16)."""

    def __init__(self, sess, d_in: int, d_out: int, rank: int, n_adapters: int, max_rows: int, buffer_tokens: int,
                 seed: int = 0):
        import torch
        from . import binding as mb
        self.torch, self.mb, self.sess = torch, mb, sess
        w = synth.Workload("coserve", d_in, d_out, rank, n_adapters, "bf16", max_rows,
                           synth.segments_array([(0, max_rows, 0, 0)]), seed=seed)
        t = synth.make_tensors(w, with_grad=False)
        dev = sess.device
        self.W, self.A, self.B, self.X = (sess.to_device(t[k], "bf16") for k in ("W", "A_all", "B_all", "X"))
        self.scale = torch.from_numpy(t["scale"]).to(dev)
        self.layer = mb.make_layer(self.W, self.A, self.B, self.scale)
        self.Y = torch.empty((max_rows, d_out), dtype=torch.bfloat16, device=dev)
        self.x_save = torch.empty((buffer_tokens, d_in), dtype=torch.bfloat16, device=dev)
        self.u_save = torch.empty((buffer_tokens, rank), dtype=torch.float32, device=dev)
        self.dY = sess.to_device(synth.normal(seed, 77, buffer_tokens * d_out).reshape(buffer_tokens, d_out), "bf16")
        self.dX = torch.empty((buffer_tokens, d_in), dtype=torch.bfloat16, device=dev)
        self.n_adapters, self.rank, self.d_in, self.d_out, self.cap = n_adapters, rank, d_in, d_out, buffer_tokens
        self.opt: Dict[int, list] = {}
        self.step_no = 0
        self.dA = self.dB = None
        self.slots: List[int] = []

    def forward(self, table, n_rows, save_base, cancel=False) -> bool:
        mb = self.mb
        plan = mb.mlora_plan_create_async(self.sess.ctx, table, n_rows, self.n_adapters)
        try:
            if cancel:
                return False
            mb.mlora_mixed_forward(self.sess.ctx, self.layer, plan, self.X, self.Y, self.x_save, self.u_save, save_base,
                                   self.cap)
        finally:
            mb.mlora_plan_release(plan)
        return True

    def backward(self, table, n_rows) -> None:
        mb, torch = self.mb, self.torch
        plan = mb.mlora_plan_create_async(self.sess.ctx, table, n_rows, self.n_adapters)
        try:
            self.slots = mb.mlora_plan_ft_adapters(plan)
            n = max(len(self.slots), 1)
            self.dA = torch.empty((n, self.rank, self.d_in), dtype=torch.float32, device=self.sess.device)
            self.dB = torch.empty((n, self.rank, self.d_out), dtype=torch.float32, device=self.sess.device)
            mb.mlora_backward(self.sess.ctx, self.layer, plan, self.dY, self.x_save, self.u_save, self.dA, self.dB, self.dX)
        finally:
            mb.mlora_plan_release(plan)

    def update(self, table, n_rows) -> None:
        mb, torch = self.mb, self.torch
        plan = mb.mlora_plan_create_async(self.sess.ctx, table, n_rows, self.n_adapters)
        try:
            key = tuple(self.slots)
            if key not in self.opt:
                idx = torch.tensor(self.slots, device=self.sess.device)
                wA, wB = self.A[idx].float().contiguous(), self.B[idx].float().contiguous()
                self.opt[key] = [wA, wB] + [torch.zeros_like(x) for x in (wA, wA, wB, wB)]
            wA, wB, mA, vA, mB, vB = self.opt[key]
            self.step_no += 1
            mb.mlora_adamw_update(self.sess.ctx, self.layer, plan, self.dA, self.dB, wA, wB, mA, vA, mB, vB, self.step_no,
                                  lr=1e-6)
        finally:
            mb.mlora_plan_release(plan)


def synthetic_arrivals(n_steps: int, seed: int, n_adapters: int):
    """Per step: (prefill [(tokens, adapter)], decode adapters, kv tokens).  One step in three carries
    one to three prompts of 64-512 tokens; 64-256 requests decode."""
    u = synth.uniform01(seed, 4242, 0, 8 * n_steps)
    for i in range(n_steps):
        a = u[8 * i:8 * i + 8]
        prefill = []
        if a[0] < 1.0 / 3.0:
            for j in range(1 + int(a[1] * 3)):
                prefill.append((64 + int(a[2 + j] * 448), int(a[5] * n_adapters) % n_adapters))
        n_dec = 64 + int(a[6] * 192)
        dec = [(i + j) % n_adapters for j in range(n_dec)]
        yield prefill, dec, 512 * n_dec


def main(argv=None):
    import torch
    from . import binding as mb
    from .runner import Session
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--slack", type=float, default=1.5, help="SLO budget as a multiple of the inference-only step time")
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("the co-serving loop runs the CUDA path: no GPU visible")
    d_in, d_out, rank, n_adapters, max_rows, buf = 4096, 4096, 16, 32, 4096, 2048
    lines = []
    with Session(0) as sess:
        ex = GpuExecutor(sess, d_in, d_out, rank, n_adapters, max_rows, buf)

        def timed(fn):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(); e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        # calibration of the linear terms of Eq. I on this projection (ms): a few batch compositions
        obs = []
        loop0 = CoServeLoop(ex, None, n_adapters)
        for t_in, n_dec, ft in ((256, 0, 0), (1024, 0, 0), (2048, 256, 0), (512, 256, 256), (1024, 128, 512),
                                (0, 256, 1024), (2048, 0, 1024), (256, 64, 0), (0, 128, 0), (3072, 256, 512)):
            pre = [(t_in, 0)] if t_in else []
            ftl = [SavedSample(-1, 256, 0) for _ in range(ft // 256)]
            table, rows = loop0._step_table(pre, [0] * n_dec, ftl)
            for _ in range(2):
                ex.forward(table, rows, 0)
            tms = min(timed(lambda: ex.forward(table, rows, 0)) for _ in range(3))
            obs.append(([t_in] * bool(t_in) + [256] * (ft // 256), n_dec, 0, ft, tms))
        coef = ms.mlora_fit_mixed(obs, ms.FIT_BETA | ms.FIT_GAMMA | ms.FIT_C)
        lines.append(f"fitted on this projection (ms, includes per-step plan creation): beta {coef.beta:.3e}/token, "
                     f"gamma {coef.gamma:.3e}/ft token, c {coef.c:.3e}")

        largest = ms.mlora_predict_mixed(coef, [512, 512, 512], 256, 0, 0)      # the largest inference step of the pattern
        for slack in (None, 1.0, args.slack, 3.0):       # None: inference only (empty pool), the baseline row
            # TTFT budget of a step with prompts = slack x its predicted inference-only time (Eq. III with the
            # arrival time chosen accordingly); the TPOT SLO = slack x the largest inference step
            with_ft = slack is not None
            slack = slack if with_ft else 1.0
            sched = ms.mlora_sched_create(coef, coef, ms.decode_coef(), 1.0, slack * largest, buf)
            for i in range(64 if with_ft else 0):
                ms.mlora_sched_pool_add(sched, i, 256)
            loop = CoServeLoop(ex, sched, n_adapters, ft_adapter_of=lambda sid: sid % 4)
            n_steps = ft_tokens = inf_tokens = 0
            ms_total = 0.0
            step_ms = []
            next_id = 64
            for prefill, dec, kv in synthetic_arrivals(args.steps, 1, n_adapters):
                lens = [n for n, _ in prefill]
                budget = slack * ms.mlora_predict_mixed(coef, lens, len(dec), 0, 0)
                info = {}

                def run():
                    info.update(loop.step(prefill, dec, 0, t_now=(1.0 - budget) if lens else 0.0,
                                          earliest_arrival=0.0 if lens else None))
                step_ms.append(timed(run))
                ms_total += step_ms[-1]
                n_steps += 1
                ft_tokens += info["ft_tokens"]
                inf_tokens += sum(lens) + len(dec)
                while with_ft and ms.mlora_sched_pool_size(sched) < 32:
                    ms.mlora_sched_pool_add(sched, next_id, 256); next_id += 1
            lines.append(f"| {f'{slack:.2f}' if with_ft else 'inference only'} | {n_steps} | {np.median(step_ms):.3f} | {np.quantile(step_ms, 0.99):.3f} | "
                         f"{inf_tokens / ms_total * 1e3:.0f} | {ft_tokens / ms_total * 1e3:.0f} | {loop.n_backward} | "
                         f"{len(loop.trained)} |")
            ms.mlora_sched_destroy(sched)
    head = ["| budget / inference-only time | steps | median ms per step (incl. planning, backward, update) | p99 ms | "
            "inference tokens/s | fine-tuning tokens/s | backward passes | samples trained |", "|---|---|---|---|---|---|---|---|"]
    text = lines[0] + "\n\n" + "\n".join(head + lines[1:]) + "\n"
    sys.stdout.write(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
