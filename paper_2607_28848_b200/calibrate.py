"""Estimator calibration (Section 4.2) against this library's own forward path: times the seven
projections of one decoder layer over a grid of batch compositions and fits Eq. I's linear
coefficients (beta per input token, gamma per fine-tuning token whose activations are saved, c)
with `mlora_fit_mixed`.  The attention and KV-cache terms (alpha, eps) have no counterpart in a
projection layer and stay 0.  Then runs Algorithm 1 (`mlora_sched_admit`) with the fitted
coefficients on the layer-set batch mix to show what the fit admits.

    python -m paper_2607_28848_b200.calibrate [--steps 10] [--out table.md]

Grid, as the calibration recipe sweeps: total prefill length, its split over requests, decode
batch size, fine-tuning tokens.  Times are milliseconds of the forward of all seven projections.
"""
from __future__ import annotations

import argparse
import sys
from typing import List, Tuple

import numpy as np
import torch

from . import binding as mb
from . import sched as ms
from . import synth
from .runner import Session

MAX_ROWS = 5120
FT_SAMPLE = 256


def batch_segments(prefill_lens: List[int], n_decode: int, ft_tokens: int, n_adapters: int) -> Tuple[np.ndarray, int]:
    """Prefill requests, then decode rows, then fine-tuning samples of 256 tokens; adapters round-robin."""
    segs, row, k = [], 0, 0
    for n in prefill_lens:
        segs.append((row, n, k % n_adapters, 0)); row += n; k += 1
    for _ in range(n_decode):
        segs.append((row, 1, k % n_adapters, 0)); row += 1; k += 1
    left = ft_tokens
    while left > 0:
        n = min(FT_SAMPLE, left)
        segs.append((row, n, k % 4, 1)); row += n; left -= n; k += 1
    return synth.segments_array(segs), row


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("calibration times the CUDA path: no GPU visible")
    lines = []
    with Session(0) as sess:
        layers = []
        for w in synth.cfg3_layer_set(0):
            big = synth.Workload(w.name, w.d_in, w.d_out, w.rank, w.n_adapters, w.dtype, MAX_ROWS,
                                 synth.segments_array([(0, MAX_ROWS, 0, 0)]), seed=0, tag_base=w.tag_base)
            t = synth.make_tensors(big, with_grad=False)
            dev = {k: sess.to_device(t[k], w.dtype) for k in ("W", "A_all", "B_all", "X")}
            dev["scale"] = torch.from_numpy(t["scale"]).to(sess.device)
            dev["Y"] = torch.empty((MAX_ROWS, w.d_out), dtype=torch.bfloat16, device=sess.device)
            dev["x_save"] = torch.empty((MAX_ROWS, w.d_in), dtype=torch.bfloat16, device=sess.device)
            dev["u_save"] = torch.empty((MAX_ROWS, w.rank), dtype=torch.float32, device=sess.device)
            dev["layer"] = mb.make_layer(dev["W"], dev["A_all"], dev["B_all"], dev["scale"])
            layers.append(dev)
        n_adapters = layers[0]["A_all"].shape[0]

        grid = []
        for total in (256, 512, 1024, 2048, 3072):
            for split in (1, 4):
                for n_dec in (0, 256, 1024):
                    for ft in (0, 256, 512, 1024):
                        if total + n_dec + ft <= MAX_ROWS:
                            grid.append(([total // split] * split, n_dec, ft))
        obs = []
        for lens, n_dec, ft in grid:
            segs, rows = batch_segments(lens, n_dec, ft, n_adapters)
            plans = [mb.mlora_plan_create(sess.ctx, segs, rows, n_adapters) for _ in layers]

            def step():
                for dev, plan in zip(layers, plans):
                    mb.mlora_mixed_forward(sess.ctx, dev["layer"], plan, dev["X"], dev["Y"], dev["x_save"],
                                           dev["u_save"], 0, MAX_ROWS)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                step()
            e1.record()
            torch.cuda.synchronize()
            ms_step = e0.elapsed_time(e1) / args.steps
            for p in plans:
                mb.mlora_plan_destroy(p)
            if mb.mlora_poll_status(sess.ctx) != 0:
                raise RuntimeError("device status non-zero during calibration")
            ft_lens = [FT_SAMPLE] * (ft // FT_SAMPLE)
            obs.append((lens + ft_lens, n_dec, 0, ft, ms_step))

    coef = ms.mlora_fit_mixed(obs, ms.FIT_BETA | ms.FIT_GAMMA | ms.FIT_C)
    rel = []
    for lens, n_dec, kv, ft, t in obs:
        pred = ms.mlora_predict_mixed(coef, lens, n_dec, kv, ft)
        rel.append(abs(pred - t) / t)
    rel = np.asarray(rel)
    lines.append(f"observations: {len(obs)} batch compositions, forward of 7 projections, {args.steps} timed steps each")
    lines.append(f"fit (ms): beta = {coef.beta:.6e} per input token, gamma = {coef.gamma:.6e} per fine-tuning token, "
                 f"c = {coef.c:.6e}; alpha = eps = 0 (no attention / KV cache in this path)")
    lines.append(f"relative error of the fit: median {np.median(rel):.3f}, 90th percentile {np.quantile(rel, 0.9):.3f}, "
                 f"max {rel.max():.3f}")
    lines.append("")
    lines.append("| prefill lens | decode | ft tokens | measured ms | predicted ms |")
    lines.append("|---|---|---|---|---|")
    for lens, n_dec, kv, ft, t in obs[:: max(1, len(obs) // 24)]:
        n_inf = len(lens) - ft // FT_SAMPLE
        lines.append(f"| {n_inf} x {lens[0]} | {n_dec} | {ft} | {t:.3f} | {ms.mlora_predict_mixed(coef, lens, n_dec, kv, ft):.3f} |")

    # Algorithm 1 with the fitted coefficients: the layer-set inference mix, a pool of 256-token samples
    lines.append("")
    lines.append("| budget ms | admitted samples | admitted tokens | predicted step ms |")
    lines.append("|---|---|---|---|")
    inf_lens = list(synth.CFG3_PREFILL_LENS)
    base = ms.mlora_predict_mixed(coef, inf_lens, 1024, 0, 0)
    for mult in (1.0, 1.25, 1.5, 2.0, 3.0):
        s = ms.mlora_sched_create(coef, coef, ms.decode_coef(), base * mult, 1e9, 8192)
        for i in range(32):
            ms.mlora_sched_pool_add(s, i, FT_SAMPLE)
        ids, toks, budget = ms.mlora_sched_admit(s, inf_lens, 1024, 0, 0.0, 0.0)
        pred = ms.mlora_predict_mixed(coef, inf_lens + toks, 1024, 0, sum(toks))
        ms.mlora_sched_destroy(s)
        lines.append(f"| {budget:.3f} | {len(ids)} | {sum(toks)} | {pred:.3f} |")
    text = "\n".join(lines) + "\n"
    sys.stdout.write(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
