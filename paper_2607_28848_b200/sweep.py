"""Rank / adapter-count / fine-tune-fraction sweep on the 4096 -> 14336 projection (2048 rows,
Zipf(1.1) adapter popularity): forward + LoRA backward per point, timed with CUDA events.

    python -m paper_2607_28848_b200.sweep [--ranks 8,16,...] [--adapters 1,8,64,256] [--fractions 0,0.25,0.5,0.75]
                                          [--unsorted] [--steps 20] [--out table.md]

Prints a markdown table: ms per forward+backward, tokens/s, TFLOP/s (algorithmic FLOPs) and the
fraction of the measured bf16 peak.  W and X are drawn once per run; adapters per (rank, count).
"""
from __future__ import annotations

import argparse
import sys

import numpy as np
import torch

from . import synth
from .accounting import flops, load_peaks
from .runner import LayerRun, Session


def run_point(sess, w, tensors, steps: int, warmup: int = 3):
    run = LayerRun(sess, w.dtype, tensors, w.segments, w.n_rows)
    has_ft = run.ft_rows > 0

    def step():
        run.forward()
        if has_ft:
            run.backward()
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    status = run.status()
    run.close()
    if status != 0:
        raise RuntimeError(f"device status {status} at {w.name}")
    return ms


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--ranks", default="8,16,32,64,128")
    ap.add_argument("--adapters", default="1,8,64,256")
    ap.add_argument("--fractions", default="0,0.25,0.5,0.75")
    ap.add_argument("--unsorted", action="store_true", help="every inference row its own segment, rows not sorted by adapter")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    ranks = [int(x) for x in args.ranks.split(",")]
    counts = [int(x) for x in args.adapters.split(",")]
    fracs = [float(x) for x in args.fractions.split(",")]
    peaks = load_peaks()
    lines = [f"| rank | adapters | ft fraction | segments | ms fwd+bwd | M tokens/s | TFLOP/s | of burst peak ({peaks['bf16_tflops']:.0f}) |",
             "|---|---|---|---|---|---|---|---|"]
    with Session(0) as sess:
        base = synth.cfg4_sweep_point(ranks[0], counts[0], fracs[0])
        shared = synth.make_tensors(base)                    # X, W, dY shapes do not depend on rank / count
        for r in ranks:
            for n in counts:
                w0 = synth.cfg4_sweep_point(r, n, 0.0)
                ad = synth.make_tensors(w0, with_grad=False)
                for f in fracs:
                    w = synth.cfg4_sweep_point(r, n, f, sorted_rows=not args.unsorted)
                    t = {"X": shared["X"], "W": shared["W"], "A_all": ad["A_all"], "B_all": ad["B_all"],
                         "scale": ad["scale"]}
                    if w.ft_rows:
                        t["dY"] = synth.round_to_bf16(synth.normal(0, 5, w.ft_rows * w.d_out).reshape(w.ft_rows, w.d_out))
                    ms = run_point(sess, w, t, args.steps)
                    fl = flops(w)
                    tot = fl["fwd"] + (fl["bwd"] if w.ft_rows else 0.0)
                    tf = tot / ms / 1e9
                    lines.append(f"| {r} | {n} | {f:g} | {len(w.segments)} | {ms:.3f} | {w.n_rows / ms / 1e3:.2f} | {tf:.0f} | "
                                 f"{tf / peaks['bf16_tflops']:.2f} |")
                    print(lines[-1], flush=True)
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as fh:
            fh.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
