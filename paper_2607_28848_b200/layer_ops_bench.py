"""Throughput of the layer pieces (RMSNorm, rotary embedding, SiLU gate, add; attention for a 512-token
sequence) at Llama-3-8B sizes, against the measured HBM copy bandwidth.

    python -m paper_2607_28848_b200.layer_ops_bench [--out table.md]
"""
from __future__ import annotations

import argparse
import sys

import torch

from . import layer_ops as mo
from .accounting import load_peaks


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
    return e0.elapsed_time(e1) / n * 1e-3


def whole_layer(dev) -> str:
    """One Llama-3-8B-sized decoder layer through DecoderLayer: the mixed serving forward of the cfg3 batch
    (4096 rows: 12 prompts, 1024 decode rows, four 512-token fine-tuning sequences) and the backward that
    recomputes the layer for the 2048 fine-tuning rows from the saved layer input."""
    import math
    import numpy as np
    from . import synth
    from .layer import DecoderLayer
    from .runner import Session
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
    return (f"whole decoder layer (Llama-3-8B sizes, cfg3 batch: {T} rows, {ft_rows} fine-tuning), through DecoderLayer with "
            f"PyTorch autograd stringing the kernels together (host overheads included): serving forward "
            f"{np.median(tf):.2f} ms, recompute + backward over the fine-tuning rows {np.median(tb):.2f} ms")


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="")
    ap.add_argument("--attention-only", action="store_true", help="only the attention timings (a small case for profiling)")
    args = ap.parse_args(argv)
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
        t = timeit(fn)
        lines.append(f"| {name} | {nbytes / 1e6:.0f} MB | {t * 1e6:.1f} | {nbytes / t / 1e9:.0f} | {nbytes / t / 1e9 / hbm:.2f} |")
    # attention: 4 sequences of 512 tokens, 32 query heads over 8 kv heads
    Ta = 2048
    q = torch.randn(Ta, H * dh, device=dev).to(bf)
    k, v = (torch.randn(Ta, Hkv * dh, device=dev).to(bf) for _ in range(2))
    o, dq = torch.empty_like(q), torch.empty_like(q)
    dk, dv = torch.empty_like(k), torch.empty_like(v)
    lse = torch.empty(Ta, H, device=dev)
    ss = (torch.arange(Ta, device=dev, dtype=torch.int32) // 512) * 512
    se = ss + 512
    tf = timeit(lambda: mo.mlora_attention_forward(q, k, v, o, lse, ss, se, H, Hkv, dh), n=20)
    tb = timeit(lambda: mo.mlora_attention_backward(q, k, v, o, lse, q, dq, dk, dv, ss, se, H, Hkv, dh), n=5)
    fl = 4 * 512 * 513 / 2 * dh * 2 * 2 * H               # QK^T and PV over the causal half, 4 sequences
    lines.append("")
    lines.append(f"attention, 4 sequences x 512 tokens, 32 query / 8 key-value heads of 128: forward (tcgen05 kernel) "
                 f"{tf * 1e3:.3f} ms ({fl / tf / 1e12:.1f} TFLOP/s over the causal half), backward {tb * 1e3:.2f} ms "
                 f"({2.5 * fl / tb / 1e12:.1f} TFLOP/s)")
    if not args.attention_only:
        lines += ["", whole_layer(dev)]
    text = "\n".join(lines) + "\n"
    sys.stdout.write(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
