#!/usr/bin/env python
"""Secondary measurement tables of the mixed-batch multi-LoRA layer (bench.py holds the headline step).

    python bench_tables.py cold        [--reps 60] [--copies 6] [--out table.md]
        skinny kernels cold (rotating inputs) on their largest instances, and the three cfg5 runs
    python bench_tables.py sweep       [--ranks ..] [--adapters ..] [--fractions ..] [--unsorted] [--steps 20] [--out ..]
        rank / adapter-count / fine-tune-fraction sweep on the 4096 -> 14336 projection (cfg4)
    python bench_tables.py smallbatch  [--out ..]
        256-row batches with a 256- or 512-token fine-tuning batch, with and without the K split
    python bench_tables.py layer-ops   [--attention-only] [--out ..]
        the layer pieces around the projections at Llama-3-8B sizes, and one whole decoder layer

Every table is timed with CUDA events on the launching stream after warm-up; bench.py imports
`cold_skinny`, `step_time` and `run_point` for the `configs` block of its JSON line.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2607_28848_b200 import accounting  # noqa: E402
from paper_2607_28848_b200 import binding as mb  # noqa: E402
from paper_2607_28848_b200 import synth  # noqa: E402
from paper_2607_28848_b200.accounting import flops, load_peaks  # noqa: E402
from paper_2607_28848_b200.runner import LayerRun, Session  # noqa: E402

KIND_SHRINK, KIND_GEMM_FWD, KIND_GEMM_BWD, KIND_GRAD, KIND_REDUCE = 0, 1, 2, 3, 6


def _emit(lines, out):
    text = "\n".join(lines) + "\n"
    sys.stdout.write(text)
    if out:
        with open(out, "w") as f:
            f.write(text)


def timeit(fn, n=50):
    """Mean time of fn in microseconds over n calls after 5 warm-up calls."""
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


# ---------------------------------------------------------------------------------------------
# cold skinny kernels and the three cfg5 runs
# ---------------------------------------------------------------------------------------------
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
    mb.mlora_profile_enable(sess.ctx, 16)

    def by_kind(kinds, ms, kind):
        """Launches of one kind summed: the tcgen05 families take two launches for a shrink (stream + finish) and two
        for the gradients (operand split + gradient kernel)."""
        return float(sum(m for k, m in zip(kinds.tolist(), ms.tolist()) if k == kind)) * 1e3

    try:
        for i in range(reps):
            c = i % copies
            mb.mlora_mixed_forward(sess.ctx, run.layer, run.plan, Xs[c], run.Y, xss[c], uss[c], 0, run.capacity)
            kinds, ms = mb.mlora_profile_collect(sess.ctx, 16)      # shrink (one or two launches), GEMM (and its K-split reduction, if any)
            assert kinds[0] == KIND_SHRINK and set(kinds.tolist()) <= {KIND_SHRINK, KIND_GEMM_FWD, KIND_REDUCE}, kinds
            out["shrink_fwd"].append(by_kind(kinds, ms, KIND_SHRINK))
            mb.mlora_backward(sess.ctx, run.layer, run.plan, dYs[c], xss[c], uss[c], run.dA, run.dB, run.dX)
            kinds, ms = mb.mlora_profile_collect(sess.ctx, 16)      # shrink, gradients, GEMM (and its reduction)
            assert kinds[0] == KIND_SHRINK and set(kinds.tolist()) <= {KIND_SHRINK, KIND_GRAD, KIND_GEMM_BWD, KIND_REDUCE}, kinds
            out["shrink_bwd"].append(by_kind(kinds, ms, KIND_SHRINK))
            out["grad"].append(by_kind(kinds, ms, KIND_GRAD))
    finally:
        mb.mlora_profile_enable(sess.ctx, 0)
    if run.status() != mb.MLORA_OK:
        raise RuntimeError("device status non-zero")
    run.close()
    b = accounting.algorithmic_bytes(w)
    nbytes = {"shrink_fwd": b["shrink_fwd"], "shrink_bwd": b["shrink_bwd"], "grad": b["grad_dB"] + b["grad_dA"]}
    moved = sum(x.numel() * x.element_size() for x in (Xs[0], dYs[0], xss[0]))
    return out, nbytes, moved * copies


def step_time(sess, w, reps, tensors=None, adapter_rank=None):
    """Median and best time (µs) of forward + backward (forward only without fine-tuning rows); `adapter_rank`
    makes the plan with the adapters' own ranks."""
    if tensors is None:
        tensors = synth.make_tensors(w, with_grad=w.ft_rows > 0)
    run = LayerRun(sess, w.dtype, tensors, w.segments, w.n_rows, adapter_rank=adapter_rank)

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


def table_cold(args):
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
    _emit(lines, args.out)



# ---------------------------------------------------------------------------------------------
# cfg4 sweep
# ---------------------------------------------------------------------------------------------
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


def table_sweep(args):
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
    if args.out:
        with open(args.out, "w") as fh:
            fh.write("\n".join(lines) + "\n")



# ---------------------------------------------------------------------------------------------
# small batches
# ---------------------------------------------------------------------------------------------
def table_smallbatch(args):
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
        # decode-sized forward calls: back to back (launch overlap on), and each kernel with its own event pair
        lines += ["", "| projection | decode rows | µs per forward call back to back | weight read once at the measured copy bandwidth | shrink / GEMM / reduction (event pairs) |",
                  "|---|---|---|---|---|"]
        hbm = load_peaks()["hbm_gbs"]
        names = {KIND_SHRINK: "shrink", KIND_GEMM_FWD: "gemm", KIND_REDUCE: "reduce"}
        for rows, d_in, d_out, n_ad in ((16, 4096, 4096, 4), (64, 4096, 4096, 8), (256, 4096, 4096, 32), (64, 4096, 14336, 8), (64, 14336, 4096, 8)):
            w = synth.random_workload(3, d_in, d_out, 16, n_ad, rows, max_seg=8, p_decode=0.9, p_finetune=0.0)
            run = LayerRun(sess, w.dtype, synth.make_tensors(w), w.segments, w.n_rows)
            t_call = timeit(run.forward, n=200)
            mb.mlora_profile_enable(sess.ctx, 64)
            acc = {}
            for _ in range(10):
                run.forward()
                torch.cuda.synchronize()
                kinds, ms = mb.mlora_profile_collect(sess.ctx, 32)
                for k, m in zip(kinds, ms):
                    acc.setdefault(int(k), []).append(float(m) * 1e3)
            mb.mlora_profile_enable(sess.ctx, 0)
            parts = " / ".join(f"{np.median(acc[k]):.1f}" if k in acc else "—" for k in (KIND_SHRINK, KIND_GEMM_FWD, KIND_REDUCE))
            run.close()
            lines.append(f"| {d_in} → {d_out} | {rows} | {t_call:.1f} | {d_in * d_out * 2 / hbm / 1e3:.1f} | {parts} |")
    _emit(lines, args.out)



# ---------------------------------------------------------------------------------------------
# layer pieces
# ---------------------------------------------------------------------------------------------
def whole_layer(dev) -> str:
    """One Llama-3-8B-sized decoder layer through DecoderLayer: the mixed serving forward of the cfg3 batch
    (4096 rows: 12 prompts, 1024 decode rows, four 512-token fine-tuning sequences) and the backward that
    recomputes the layer for the 2048 fine-tuning rows from the saved layer input."""
    import math
    from paper_2607_28848_b200.layer import DecoderLayer
    d, ffn, r, n_ad, H, Hkv = 4096, 14336, 16, 32, 32, 8
    dh = d // H
    g = torch.Generator().manual_seed(5)
    dims = {"q": (d, d), "k": (d, Hkv * dh), "v": (d, Hkv * dh), "o": (d, d), "gate": (d, ffn), "up": (d, ffn), "down": (ffn, d)}
    p = {"g1": torch.ones(d), "g2": torch.ones(d)}
    for name, (di, do) in dims.items():
        p["W_" + name] = (torch.randn(di, do, generator=g) / math.sqrt(di)).to(torch.bfloat16)
        p["A_" + name] = (0.02 * torch.randn(n_ad, r, di, generator=g)).to(torch.bfloat16)
        p["B_" + name] = (0.02 * torch.randn(n_ad, r, do, generator=g)).to(torch.bfloat16)
        p["s_" + name] = torch.full((n_ad,), 2.0)
    segs, T = synth.cfg3_segments(0)
    ft_rows = int(segs[segs[:, 3] != 0, 1].sum())
    x = torch.randn(T, d, generator=g).to(torch.bfloat16).to(dev)
    dy = torch.randn(ft_rows, d, generator=g).to(torch.bfloat16).to(dev)
    with Session(0) as sess:
        layer = DecoderLayer(sess, p, H, Hkv, max_ft_rows=ft_rows)
        tf, tb = [], []
        for it in range(6):
            torch.cuda.synchronize()
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            layer.forward(x, segs)
            e1.record()
            layer.backward(dy)
            e2.record()
            torch.cuda.synchronize()
            if it >= 2:
                tf.append(e0.elapsed_time(e1)); tb.append(e1.elapsed_time(e2))
        cap = layer.capture_forward(x, segs)
        tg = []
        for it in range(8):
            torch.cuda.synchronize()
            e0, e1 = (torch.cuda.Event(enable_timing=True) for _ in range(2))
            e0.record()
            cap.replay()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                tg.append(e0.elapsed_time(e1))
        y_eager = layer.forward(x, segs)
        same = bool(torch.equal(cap.y, y_eager))
        cap.close()
        saved = list(layer.saved)
        capb = layer.capture_backward(saved)
        capb.dy.copy_(dy)
        tgb = []
        for it in range(8):
            torch.cuda.synchronize()
            e0, e1 = (torch.cuda.Event(enable_timing=True) for _ in range(2))
            e0.record()
            capb.replay()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                tgb.append(e0.elapsed_time(e1))
        capb.close()
    return (f"whole decoder layer (Llama-3-8B sizes, cfg3 batch: {T} rows, {ft_rows} fine-tuning), through DecoderLayer (one "
            f"library call after the other from Python, host overheads included): serving forward "
            f"{np.median(tf):.2f} ms, recompute + backward over the fine-tuning rows {np.median(tb):.2f} ms; the same serving "
            f"forward replayed from a CUDA graph: {np.median(tg):.2f} ms (output bit-identical to the eager one: {same}); the recompute + "
            f"backward replayed from a CUDA graph: {np.median(tgb):.2f} ms")


def table_layer_ops(args):
    from paper_2607_28848_b200 import layer_ops as mo
    if not torch.cuda.is_available():
        raise RuntimeError("needs the CUDA path: no GPU visible")
    dev, bf = "cuda:0", torch.bfloat16
    hbm = load_peaks()["hbm_gbs"]
    T, d, ffn, H, Hkv, dh = 16384, 4096, 14336, 32, 8, 128          # 16384 rows: buffers larger than the L2
    x, y, dy = (torch.randn(T, d, device=dev).to(bf) for _ in range(3))
    gain = torch.ones(d, device=dev)
    pos = torch.arange(T, dtype=torch.int32, device=dev) % 512
    g, u, m = (torch.randn(T, ffn, device=dev).to(bf) for _ in range(3))
    dg, du = torch.empty_like(g), torch.empty_like(u)
    rows = [
        ("RMSNorm forward", lambda: mo.mlora_rmsnorm_forward(x, gain, y), 2 * T * d * 2),
        ("RMSNorm backward", lambda: mo.mlora_rmsnorm_backward(x, gain, dy, y), 3 * T * d * 2),
        ("rotary embedding (32 heads)", lambda: mo.mlora_rope(x, y, pos, H, dh), 2 * T * d * 2),
        ("SiLU gate forward", lambda: mo.mlora_swiglu_forward(g, u, m), 3 * T * ffn * 2),
        ("SiLU gate backward", lambda: mo.mlora_swiglu_backward(g, u, m, dg, du), 5 * T * ffn * 2),
        ("add", lambda: mo.mlora_add(x, dy, y), 3 * T * d * 2),
    ]
    lines = ["| kernel | bytes | µs | GB/s | of the measured copy bandwidth |", "|---|---|---|---|---|"]
    for name, fn, nbytes in ([] if args.attention_only else rows):
        t = timeit(fn) * 1e-6
        lines.append(f"| {name} | {nbytes / 1e6:.0f} MB | {t * 1e6:.1f} | {nbytes / t / 1e9:.0f} | {nbytes / t / 1e9 / hbm:.2f} |")
    # attention: 32 query heads over 8 kv heads; the first case (4 sequences of 512 tokens) is the one the layer runs
    lines.append("")
    for n_seq, L in ((4, 512), (4, 2048), (1, 8192), (16, 128)):
        Ta = n_seq * L
        q = torch.randn(Ta, H * dh, device=dev).to(bf)
        k, v = (torch.randn(Ta, Hkv * dh, device=dev).to(bf) for _ in range(2))
        o, dq = torch.empty_like(q), torch.empty_like(q)
        dk, dv = torch.empty_like(k), torch.empty_like(v)
        lse = torch.empty(Ta, H, device=dev)
        ss = (torch.arange(Ta, device=dev, dtype=torch.int32) // L) * L
        se = ss + L
        tf = timeit(lambda: mo.mlora_attention_forward(q, k, v, o, lse, ss, se, H, Hkv, dh), n=20) * 1e-6
        tb = timeit(lambda: mo.mlora_attention_backward(q, k, v, o, lse, q, dq, dk, dv, ss, se, H, Hkv, dh), n=5) * 1e-6
        fl = n_seq * L * (L + 1) / 2 * dh * 2 * 2 * H         # QK^T and PV over the causal half
        lines.append(f"attention, {n_seq} sequences x {L} tokens, 32 query / 8 key-value heads of 128: forward (tcgen05 kernel) "
                     f"{tf * 1e3:.3f} ms ({fl / tf / 1e12:.1f} TFLOP/s over the causal half), backward {tb * 1e3:.2f} ms "
                     f"({2.5 * fl / tb / 1e12:.1f} TFLOP/s)")
        if mo.mlora_layer_ops_poll_status() != 0:
            raise RuntimeError("device status non-zero")
    if not args.attention_only:
        lines += ["", whole_layer(dev)]
    _emit(lines, args.out)




def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("table", choices=["cold", "sweep", "smallbatch", "layer-ops"])
    ap.add_argument("--out", default="")
    ap.add_argument("--reps", type=int, default=60)
    ap.add_argument("--copies", type=int, default=6)
    ap.add_argument("--ranks", default="8,16,32,64,128")
    ap.add_argument("--adapters", default="1,8,64,256")
    ap.add_argument("--fractions", default="0,0.25,0.5,0.75")
    ap.add_argument("--unsorted", action="store_true", help="every inference row its own segment, rows not sorted by adapter")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--attention-only", action="store_true", help="only the attention timings (a small case for profiling)")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("these timings need the CUDA path: no GPU visible")
    {"cold": table_cold, "sweep": table_sweep, "smallbatch": table_smallbatch, "layer-ops": table_layer_ops}[args.table](args)


if __name__ == "__main__":
    main()
