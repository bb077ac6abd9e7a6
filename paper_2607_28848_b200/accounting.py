"""Algorithmic work of the mixed-batch multi-LoRA layer (FLOPs and bytes per kernel class) and the
measured peaks they are compared with.  No credit is given for padded tiles or recomputation:
every operand counts once."""
from __future__ import annotations

import json
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def flops(w) -> dict:
    """Algorithmic FLOPs: no credit for padded tiles or recomputation."""
    T, Tf, di, do, r = w.n_rows, w.ft_rows, w.d_in, w.d_out, w.rank
    return {
        "fwd": 2.0 * T * di * do + 2.0 * T * r * (di + do),
        "bwd": 2.0 * Tf * di * do + 2.0 * Tf * r * (2 * do + 2 * di),
        "gemm_fwd": 2.0 * T * do * (di + r),          # base product + expand, one kernel
        "gemm_bwd": 2.0 * Tf * di * (do + r),         # dY W^T + V A, one kernel
    }


def algorithmic_bytes(w) -> dict:
    """Each tensor once (bytes), per kernel class."""
    T, Tf, di, do, r, e = w.n_rows, w.ft_rows, w.d_in, w.d_out, w.rank, w.elem_bytes
    seg = w.segments
    used = len(set(seg[seg[:, 2] >= 0, 2].tolist())) if len(seg) else 0
    fta = len(set(seg[seg[:, 3] != 0, 2].tolist())) if len(seg) else 0
    return {
        "shrink_fwd": e * T * di + e * used * r * di + 4 * T * r + e * Tf * di + 4 * Tf * r,   # + save copies
        "shrink_bwd": e * Tf * do + e * fta * r * do + 4 * Tf * r,
        "grad_dB": e * Tf * do + 4 * Tf * r + 4 * fta * r * do,
        "grad_dA": e * Tf * di + 4 * Tf * r + 4 * fta * r * di,
        "gemm_fwd": e * (T * di + di * do + T * do + used * r * do) + 4 * T * r,
        "gemm_bwd": e * (Tf * do + di * do + Tf * di + fta * r * di) + 4 * Tf * r,
    }


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}
