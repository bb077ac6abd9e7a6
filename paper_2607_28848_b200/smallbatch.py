"""Small-batch timings: forward and backward of one projection with 256 inference rows and a 256- or
512-token fine-tuning batch (the paper's backward batches are 256 tokens), with and without the K split
of the two-SM GEMM (kernel variant 4 switches it off).

    python -m paper_2607_28848_b200.smallbatch [--out table.md]
"""
from __future__ import annotations

import argparse
import sys

import torch

from . import binding as mb
from . import synth
from .runner import LayerRun, Session


def timeit(fn, n=50):
    for _ in range(5):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n * 1e3


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("small-batch timings need the CUDA path: no GPU visible")
    lines = ["| projection | rows (inference + fine-tune) | forward µs: no split / default | backward µs: no split / default |",
             "|---|---|---|---|"]
    with Session(0) as sess:
        for t_ft in (256, 512):
            for d_in, d_out in ((4096, 4096), (4096, 14336), (14336, 4096)):
                segs = synth.segments_array([(0, 256, 1, 0), (256, t_ft, 0, 1)])
                w = synth.Workload("small", d_in, d_out, 16, 4, "bf16", 256 + t_ft, segs)
                run = LayerRun(sess, w.dtype, synth.make_tensors(w), w.segments, w.n_rows)
                res = {}
                for path in (4, 0):
                    mb.mlora_set_gemm_path(sess.ctx, path)
                    res[path] = (timeit(run.forward), timeit(run.backward))
                mb.mlora_set_gemm_path(sess.ctx, 0)
                if run.status() != mb.MLORA_OK:
                    raise RuntimeError("device status non-zero")
                run.close()
                lines.append(f"| {d_in} → {d_out} | 256 + {t_ft} | {res[4][0]:.1f} / {res[0][0]:.1f} | {res[4][1]:.1f} / {res[0][1]:.1f} |")
    text = "\n".join(lines) + "\n"
    sys.stdout.write(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
