"""Cold timings of the skinny kernels on their largest instances, and the three cfg5 runs.

Part 1 (HBM accounting of the skinny kernels): for the cfg3 gate and down projections and for cfg5,
every repetition runs forward and backward on ANOTHER copy of X, dY and the activation buffers
(enough copies to exceed the L2 several times; the base product between two skinny launches streams
more than an L2 of weights and outputs as well), with one CUDA event pair around every launch of the
library.  Reported per kernel: median and best time over the repetitions, algorithmic bytes (every
operand once, the save copies included), bytes / time against the measured copy bandwidth.

Part 2 (cfg5): decode-only, fine-tune-only and mixed steps of the 5120 -> 13824 projection and the fill
ratio t_mixed / (t_decode + t_finetune): below 1 means the fine-tuning rows ride in the pass the decode
rows need anyway.

    python -m paper_2607_28848_b200.skinny_cold [--reps 60] [--out table.md]
"""
from __future__ import annotations

import argparse
import sys

import numpy as np
import torch

from . import accounting
from . import binding as mb
from . import synth
from .runner import LayerRun, Session

KIND_SHRINK, KIND_GEMM_FWD, KIND_GEMM_BWD, KIND_GRAD, KIND_REDUCE = 0, 1, 2, 3, 6


def cold_skinny(sess, w, reps, copies):
    """Per-launch times (µs) of the shrink and gradient kernels of one projection, inputs rotated."""
    t = synth.make_tensors(w)
    run = LayerRun(sess, w.dtype, t, w.segments, w.n_rows)
    Xs = [run.X] + [run.X.clone() for _ in range(copies - 1)]
    dYs = [run.dY] + [run.dY.clone() for _ in range(copies - 1)]
    xss = [run.x_save] + [torch.empty_like(run.x_save) for _ in range(copies - 1)]
    uss = [run.u_save] + [torch.empty_like(run.u_save) for _ in range(copies - 1)]
    for i in range(copies):            # every activation buffer holds a valid forward before the timed loop
        mb.mlora_mixed_forward(sess.ctx, run.layer, run.plan, Xs[i], run.Y, xss[i], uss[i], 0, run.capacity)
    for _ in range(3):
        run.forward(); run.backward()
    torch.cuda.synchronize()
    out = {"shrink_fwd": [], "shrink_bwd": [], "grad": []}
    mb.mlora_profile_enable(sess.ctx, 8)
    try:
        for i in range(reps):
            c = i % copies
            mb.mlora_mixed_forward(sess.ctx, run.layer, run.plan, Xs[c], run.Y, xss[c], uss[c], 0, run.capacity)
            kinds, ms = mb.mlora_profile_collect(sess.ctx, 16)      # shrink, GEMM (and its K-split reduction, if any)
            assert kinds[0] == KIND_SHRINK and set(kinds[1:].tolist()) <= {KIND_GEMM_FWD, KIND_REDUCE}, kinds
            out["shrink_fwd"].append(ms[0] * 1e3)
            mb.mlora_backward(sess.ctx, run.layer, run.plan, dYs[c], xss[c], uss[c], run.dA, run.dB, run.dX)
            kinds, ms = mb.mlora_profile_collect(sess.ctx, 16)      # shrink, gradients, GEMM (and its reduction)
            assert kinds[0] == KIND_SHRINK and kinds[1] == KIND_GRAD and set(kinds[2:].tolist()) <= {KIND_GEMM_BWD, KIND_REDUCE}, kinds
            out["shrink_bwd"].append(ms[0] * 1e3)
            out["grad"].append(ms[1] * 1e3)
    finally:
        mb.mlora_profile_enable(sess.ctx, 0)
    if run.status() != mb.MLORA_OK:
        raise RuntimeError("device status non-zero")
    run.close()
    b = accounting.algorithmic_bytes(w)
    nbytes = {"shrink_fwd": b["shrink_fwd"], "shrink_bwd": b["shrink_bwd"], "grad": b["grad_dB"] + b["grad_dA"]}
    moved = sum(x.numel() * x.element_size() for x in (Xs[0], dYs[0], xss[0]))
    return out, nbytes, moved * copies


def step_time(sess, w, reps):
    """Median and best time (µs) of forward + backward (forward only without fine-tuning rows)."""
    run = LayerRun(sess, w.dtype, synth.make_tensors(w, with_grad=w.ft_rows > 0), w.segments, w.n_rows)

    def step():
        run.forward()
        if w.ft_rows:
            run.backward()

    for _ in range(5):
        step()
    torch.cuda.synchronize()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=sess.device)
    times = []
    for _ in range(reps):
        flush.zero_()                  # nothing of the previous repetition survives in the L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); step(); e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    if run.status() != mb.MLORA_OK:
        raise RuntimeError("device status non-zero")
    run.close()
    return float(np.median(times)), float(np.min(times))


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=60)
    ap.add_argument("--copies", type=int, default=6)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("these timings need the CUDA path: no GPU visible")
    peaks = accounting.load_peaks()
    hbm = peaks["hbm_gbs"]
    lines = [f"copy bandwidth used as the denominator: {hbm:.0f} GB/s ({peaks['source']}); {args.reps} repetitions, "
             f"{args.copies} rotating copies of X, dY and the activation buffers", "",
             "| workload | kernel | algorithmic MB | median µs | best µs | GB/s (median) | of the copy bandwidth (median / best) |",
             "|---|---|---|---|---|---|---|"]
    with Session(0) as sess:
        work = synth.cfg3_layer_set(0, projections=["gate", "down"]) + [synth.cfg5_decode_heavy(0)]
        for w in work:
            out, nbytes, rotated = cold_skinny(sess, w, args.reps, args.copies)
            names = {"shrink_fwd": "shrink forward (U, activation save, operand chunks)",
                     "shrink_bwd": "shrink backward (V)", "grad": "gradients (dB and dA, one launch)"}
            for k in ("shrink_fwd", "shrink_bwd", "grad"):
                med, best = float(np.median(out[k])), float(np.min(out[k]))
                lines.append(f"| {w.name} ({rotated / 1e6:.0f} MB rotated) | {names[k]} | {nbytes[k] / 1e6:.1f} | {med:.1f} | "
                             f"{best:.1f} | {nbytes[k] / med / 1e3:.0f} | {nbytes[k] / med / 1e3 / hbm:.2f} / "
                             f"{nbytes[k] / best / 1e3 / hbm:.2f} |")
        lines += ["", "| cfg5 run | rows | median µs | best µs |", "|---|---|---|---|"]
        t = {}
        for mode in ("decode", "finetune", "mixed"):
            w = synth.cfg5_decode_heavy(0, mode)
            t[mode] = step_time(sess, w, args.reps)
            lines.append(f"| {mode} | {w.n_rows} ({w.ft_rows} fine-tune) | {t[mode][0]:.1f} | {t[mode][1]:.1f} |")
        lines += ["", f"fill ratio t_mixed / (t_decode + t_finetune) = {t['mixed'][0] / (t['decode'][0] + t['finetune'][0]):.3f} "
                      f"(medians), {t['mixed'][1] / (t['decode'][1] + t['finetune'][1]):.3f} (best times)"]
    text = "\n".join(lines) + "\n"
    sys.stdout.write(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
