"""Seeded synthetic inputs for the mixed-batch multi-LoRA layer.

This module only *draws numbers and lays out segment tables*.  It contains none of
the method's arithmetic (no products, no gradients) so that both the CPU oracle's
tests and the CUDA path's tests can be fed from it without sharing any logic.

The inputs stand in for the paper's workload (a Llama-3-8B-shaped model with LoRA
adapters of rank 16 and scaling 32, Section 5 "Fine-tuning Workload"; batches that
mix inference prefill/decode tokens with fine-tuning tokens, Section 3.2 "Mixed
forward batch").  Model weights, the instruction-tuning corpus and the production
trace are replaced by Gaussian tensors and hand-listed segment mixes of the same
shapes.

Everything is produced by one counter-based generator: element ``i`` of the tensor
with tag ``g`` under seed ``s`` is a pure function of ``(s, g, i)``, so a tensor can
be regenerated piecewise and independently of any other.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_U64 = np.uint64
_MASK = (1 << 64) - 1


# --------------------------------------------------------------------------------------
# counter-based random numbers
# --------------------------------------------------------------------------------------
def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on an array of uint64 (wrapping arithmetic)."""
    z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
    return z ^ (z >> _U64(31))


def _stream_key(seed: int, tag: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + tag * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK
    # one scalar round of the same finaliser, done with Python ints
    k = ((k ^ (k >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    k = ((k ^ (k >> 27)) * 0x94D049BB133111EB) & _MASK
    return k ^ (k >> 31)


def uniform_bits(seed: int, tag: int, start: int, count: int) -> np.ndarray:
    """``count`` uint64 words for counters ``start .. start+count-1`` of stream (seed, tag)."""
    key = _U64(_stream_key(seed, tag))
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + count, dtype=np.uint64)
        return _mix64(ctr * _U64(0x9E3779B97F4A7C15) + key)


def uniform01(seed: int, tag: int, start: int, count: int) -> np.ndarray:
    """Uniform doubles in (0, 1)."""
    bits = uniform_bits(seed, tag, start, count)
    return ((bits >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, tag: int, count: int, std: float = 1.0, chunk: int = 1 << 22) -> np.ndarray:
    """``count`` independent N(0, std^2) float64 draws (Box-Muller on counter pairs).

    Every element is a function of (seed, tag, index) alone, so the chunks are independent; large
    draws spread them over the host's cores (numpy releases the interpreter lock inside its loops).
    """
    out = np.empty(count, dtype=np.float64)

    def fill(lo: int) -> None:
        n = min(chunk, count - lo)
        u1 = uniform01(seed, tag, 2 * lo, 2 * n)
        u2 = u1[1::2]
        u1 = u1[0::2]
        out[lo:lo + n] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        if std != 1.0:
            out[lo:lo + n] *= std

    starts = range(0, count, chunk)
    if len(starts) > 1:
        import os
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(len(starts), os.cpu_count() or 1)) as pool:
            list(pool.map(fill, starts))
    else:
        for lo in starts:
            fill(lo)
    return out


def randint(seed: int, tag: int, count: int, high: int) -> np.ndarray:
    """``count`` integers uniform in [0, high)."""
    return (uniform01(seed, tag, 0, count) * high).astype(np.int64).clip(0, high - 1)


# --------------------------------------------------------------------------------------
# storage rounding (inputs are rounded ONCE here; both sides then see identical values)
# --------------------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); returned as float32."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32).reshape(f.shape)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(f"unknown storage dtype {dtype!r}")


# --------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------
SEG_DTYPE = np.int32  # rows of (row_start, row_len, adapter_id, is_finetune)


@dataclass
class Workload:
    """One projection with one mixed batch.

    ``segments`` is an int32 array [n_seg, 4] of (row_start, row_len, adapter_id,
    is_finetune).  Rows not covered by a segment, and segments with adapter -1, use
    the base weight only.
    """
    name: str
    d_in: int
    d_out: int
    rank: int
    n_adapters: int
    dtype: str            # "bf16" or "f32": storage type of X, W, A, B, Y, dY, dX
    n_rows: int
    segments: np.ndarray
    lora_scale: float = 2.0       # alpha / r = 32 / 16 (Section 5, "Fine-tuning Workload")
    seed: int = 0
    tag_base: int = 0             # keeps projections of one layer set on distinct streams
    notes: str = ""

    @property
    def ft_rows(self) -> int:
        s = self.segments
        return int(s[s[:, 3] != 0, 1].sum()) if len(s) else 0

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


def segments_array(segs: Sequence[Sequence[int]]) -> np.ndarray:
    a = np.asarray(list(segs), dtype=SEG_DTYPE).reshape(-1, 4)
    return np.ascontiguousarray(a)


def layout_segments(prefill: Sequence[Tuple[int, int]], decode: Sequence[int],
                    finetune: Sequence[Tuple[int, int]]) -> Tuple[np.ndarray, int]:
    """Measurement row order: prefill segments, then decode rows, then fine-tune segments.

    ``prefill`` / ``finetune`` are (length, adapter) pairs, ``decode`` is one adapter id per
    single-token row.  Returns (segment table, total rows).
    """
    segs: List[Tuple[int, int, int, int]] = []
    row = 0
    for ln, ad in prefill:
        segs.append((row, ln, ad, 0))
        row += ln
    for ad in decode:
        segs.append((row, 1, int(ad), 0))
        row += 1
    for ln, ad in finetune:
        segs.append((row, ln, ad, 1))
        row += ln
    return segments_array(segs), row


def make_tensors(w: Workload, with_grad: bool = True) -> Dict[str, np.ndarray]:
    """Draw X, W, A_all, B_all, scale (and dY for the fine-tune rows) for a workload.

    Distributions (second parameter read as a standard deviation):
    X ~ N(0,1), dY ~ N(0,1), W ~ N(0, d_in^-1/2), A, B ~ N(0, 0.02).  Values are rounded
    once to the storage dtype and returned as float32 arrays holding exactly those values.
    Layouts: X [n_rows, d_in]; W [d_in, d_out]; A_all [n_adapters, rank, d_in];
    B_all [n_adapters, rank, d_out]; scale [n_adapters]; dY [ft_rows, d_out].
    """
    t = w.tag_base
    out: Dict[str, np.ndarray] = {}
    out["X"] = round_to_storage(normal(w.seed, t + 1, w.n_rows * w.d_in).reshape(w.n_rows, w.d_in), w.dtype)
    out["W"] = round_to_storage(
        normal(w.seed, t + 2, w.d_in * w.d_out, std=w.d_in ** -0.5).reshape(w.d_in, w.d_out), w.dtype)
    out["A_all"] = round_to_storage(
        normal(w.seed, t + 3, w.n_adapters * w.rank * w.d_in, std=0.02).reshape(w.n_adapters, w.rank, w.d_in),
        w.dtype)
    out["B_all"] = round_to_storage(
        normal(w.seed, t + 4, w.n_adapters * w.rank * w.d_out, std=0.02).reshape(w.n_adapters, w.rank, w.d_out),
        w.dtype)
    out["scale"] = np.full(w.n_adapters, w.lora_scale, dtype=np.float32)
    if with_grad:
        n = w.ft_rows
        out["dY"] = round_to_storage(normal(w.seed, t + 5, n * w.d_out).reshape(n, w.d_out), w.dtype)
    return out


# ---- the five seeded configurations ---------------------------------------------------
def cfg1_tiny(seed: int = 0) -> Workload:
    """Tiny fp32 layer: 256 -> 256, 4 adapters of rank 8, 64 rows, one fine-tune segment."""
    segs = segments_array([(0, 24, 0, 0), (24, 16, 1, 0), (40, 8, 2, 0), (48, 16, 3, 1)])
    return Workload("cfg1_tiny", 256, 256, 8, 4, "f32", 64, segs, seed=seed)


CFG2_PREFILL_LENS = (64, 71, 97, 130, 161, 181, 64, 256)           # sums to 1024
CFG3_PREFILL_LENS = (17, 33, 64, 65, 80, 96, 99, 112, 127, 128, 101, 102)  # sums to 1024


def cfg2_single_projection(seed: int = 0) -> Workload:
    """4096 -> 4096 bf16, 16 adapters of rank 16; 1024 prefill + 64 decode + 2x256 fine-tune rows."""
    pre_ad = randint(seed, 101, len(CFG2_PREFILL_LENS), 14)
    dec_ad = randint(seed, 102, 64, 16)
    segs, rows = layout_segments(list(zip(CFG2_PREFILL_LENS, pre_ad.tolist())), dec_ad.tolist(),
                                 [(256, 14), (256, 15)])
    assert rows == 1600
    return Workload("cfg2_proj4096", 4096, 4096, 16, 16, "bf16", rows, segs, seed=seed)


CFG3_PROJECTIONS = (  # name, d_in, d_out   (Llama-3-8B shapes)
    ("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
    ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096),
)


def cfg3_segments(seed: int = 0) -> Tuple[np.ndarray, int]:
    pre_ad = randint(seed, 201, len(CFG3_PREFILL_LENS), 28)
    dec_ad = randint(seed, 202, 1024, 32)
    return layout_segments(list(zip(CFG3_PREFILL_LENS, pre_ad.tolist())), dec_ad.tolist(),
                           [(512, 28), (512, 29), (512, 30), (512, 31)])


def cfg3_layer_set(seed: int = 0, projections: Optional[Sequence[str]] = None) -> List[Workload]:
    """The seven projections of one decoder layer, each with fresh X / dY, sharing one batch mix."""
    segs, rows = cfg3_segments(seed)
    assert rows == 4096
    out = []
    for i, (name, di, do) in enumerate(CFG3_PROJECTIONS):
        if projections is not None and name not in projections:
            continue
        out.append(Workload(f"cfg3_{name}", di, do, 16, 32, "bf16", rows, segs, seed=seed,
                            tag_base=1000 * (i + 1)))
    return out


def zipf_adapters(seed: int, tag: int, count: int, n: int, exponent: float = 1.1) -> np.ndarray:
    """Adapter ids with popularity p(i) proportional to (i+1)^-exponent, truncated to n adapters."""
    p = (np.arange(1, n + 1, dtype=np.float64)) ** (-exponent)
    cdf = np.cumsum(p / p.sum())
    u = uniform01(seed, tag, 0, count)
    return np.searchsorted(cdf, u, side="right").clip(0, n - 1).astype(np.int64)


def cfg4_sweep_point(rank: int, n_adapters: int, ft_fraction: float, seed: int = 0,
                     sorted_rows: bool = True) -> Workload:
    """4096 -> 14336 bf16, 2048 rows; inference rows draw adapters from Zipf(1.1).

    Fine-tune rows come last in segments of 256 (the paper's backward batch), segment k on
    adapter k mod n.  With ``sorted_rows`` the inference rows are stably sorted by adapter and
    merged into one segment per adapter; otherwise every row is its own segment.
    """
    rows = 2048
    n_ft = int(round(rows * ft_fraction / 256.0)) * 256
    n_inf = rows - n_ft
    ad = zipf_adapters(seed, 401, n_inf, n_adapters)
    pre: List[Tuple[int, int]] = []
    dec: List[int] = []
    if sorted_rows:
        ad = np.sort(ad, kind="stable")
        if n_inf:
            cuts = np.flatnonzero(np.diff(ad)) + 1
            starts = np.concatenate(([0], cuts))
            ends = np.concatenate((cuts, [n_inf]))
            pre = [(int(e - s), int(ad[s])) for s, e in zip(starts, ends)]
    else:
        dec = ad.tolist()
    ft = [(256, k % n_adapters) for k in range(n_ft // 256)]
    segs, total = layout_segments(pre, dec, ft)
    assert total == rows
    nm = f"cfg4_r{rank}_n{n_adapters}_f{ft_fraction:g}" + ("" if sorted_rows else "_unsorted")
    return Workload(nm, 4096, 14336, rank, n_adapters, "bf16", rows, segs, seed=seed)


def cfg5_decode_heavy(seed: int = 0, mode: str = "mixed", sorted_rows: bool = False) -> Workload:
    """5120 -> 13824 bf16, 128 adapters of rank 32; 512 decode rows and/or one 2048-row fine-tune segment.

    The decode rows come in arrival order (a random adapter per row); with ``sorted_rows`` the same rows are
    ordered by adapter, the layout a serving engine that sorts its decode batch hands over."""
    dec = randint(seed, 501, 512, 128).tolist() if mode in ("mixed", "decode") else []
    if sorted_rows:
        dec = sorted(dec)
    ft = [(2048, 127)] if mode in ("mixed", "finetune") else []
    segs, rows = layout_segments([], dec, ft)
    return Workload(f"cfg5_{mode}" + ("_sorted" if sorted_rows and dec else ""), 5120, 13824, 32, 128, "bf16", rows, segs, seed=seed)


def random_workload(seed: int, d_in: int, d_out: int, rank: int, n_adapters: int, n_rows: int,
                    dtype: str = "bf16", max_seg: int = 200, p_decode: float = 0.3,
                    p_finetune: float = 0.3, p_gap: float = 0.1, p_noadapter: float = 0.1,
                    shuffle: bool = True) -> Workload:
    """A random valid table: ragged segments, single-row segments, gaps, adapter -1, any order."""
    u = uniform01(seed, 901, 0, 4 * n_rows + 8)
    segs: List[Tuple[int, int, int, int]] = []
    row, i = 0, 0
    while row < n_rows:
        a, b, c, d = u[4 * i:4 * i + 4]
        i += 1
        ln = 1 if a < p_decode else 1 + int(b * max_seg)
        ln = min(ln, n_rows - row)
        if c < p_gap:
            row += ln            # uncovered rows: base weight only
            continue
        is_ft = int(c > 1.0 - p_finetune)
        ad = int(d * n_adapters) % n_adapters
        if not is_ft and d < p_noadapter:
            ad = -1
        segs.append((row, ln, ad, is_ft))
        row += ln
    table = segments_array(segs)
    if shuffle and len(table) > 1:
        order = np.argsort(uniform01(seed, 902, 0, len(table)), kind="stable")
        table = np.ascontiguousarray(table[order])
    return Workload(f"random_s{seed}", d_in, d_out, rank, n_adapters, dtype, n_rows, table, seed=seed)
