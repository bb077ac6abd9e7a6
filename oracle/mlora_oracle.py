"""CPU oracle for the mixed-batch multi-LoRA linear layer (TEST INFRASTRUCTURE ONLY).

A plain, slow, float64 statement of what the layer computes, written from the paper's
definitions.  It exists so that the CUDA path can be checked against something that is
obviously the definition.  It shares no code with the CUDA path and must never be
imported by it: only the tests, the smoke check and the benchmark's CPU-baseline leg
may call it.

What it follows
---------------
* Section 2.2 (Parameter-Efficient Fine-Tuning): a frozen weight plus a trainable
  rank-r product, W_eff = W + B A.  In the row-vector convention used here a token
  row x maps to  y = x W + s (x A_a^T) B_a  where, per adapter a, ``A_all[a]`` is the
  paper's A (shape [r, d_in]) and ``B_all[a]`` is the transpose of the paper's B
  (shape [r, d_out]), and s_a = alpha_a / r is the LoRA scaling (Section 5, "Fine-tuning
  Workload": r = 16, alpha = 32, so s = 2).
* Section 2.2, multi-LoRA batching: rows bound to different adapters share one pass
  over the base weight, each row applying its own adapter.
* Section 3.2, "Mixed forward batch": fine-tuning rows go through exactly the same
  forward as inference rows; the only addition is that their activations are captured.
  Here the captured state is the row of X and the unscaled rank-r product x A_a^T.
* Section 3.2, "Backward subprocess": LoRA gradients are computed from the saved
  activations.  The formulas are the chain rule applied to the forward above with the
  loss gradient dY given for the fine-tuning rows:
      V  = s dY B_a^T                 [rows, r]
      dB_a += s U^T dY                [r, d_out]
      dA_a += V^T X                   [r, d_in]
      dX = dY W^T + V A_a             [rows, d_in]

Variants (Section 5, "Fine-tuning Workload": the adapter is trained with dropout 0.05; adapters of
different ranks share one base model in Section 2.2's serving setting):
* LoRA dropout acts on the input of the low-rank branch of the fine-tuning rows only (the usual
  LoRA definition: y = x W + s B A dropout(x)); inference rows never see it.  The keep decision
  of element (m, k) - m the row's place in this batch's save order, k the input column - comes
  from a counter-based generator so that forward and backward regenerate the same mask:
  output number c + 1 of the SplitMix64 stream started at ``seed``, c = m * 2^32 + (k >> 2);
  its 16-bit field number k & 3 is compared with round(p * 65536); kept elements are scaled by
  1 / (1 - p).  With the mask K (0/1) the chain rule gives U = (X * K) A^T / (1 - p),
  dA += (V / (1 - p))^T (X * K),  dX = dY W^T + (V A) * K / (1 - p); V and dB keep their form.
* Adapters of different ranks are stored padded to the layer's rank r with zero rows; a zero row of
  A_a and B_a contributes nothing to Y, V, dX and gets a zero gradient, so the padded layer
  computes exactly what the per-adapter ranks define (``forward_ragged`` states that definition).

Matrix products use numpy's float64 ``@`` as a library step; there is no blocking,
fusion or reordering beyond the definitions above.  Inputs are the stored values
(already rounded to the storage type by the caller); nothing is rounded in between.

Parity pins (tests/test_oracle_pins.py): element-by-element brute force in pure
Python on tiny shapes, a hand-computed worked example, the B = 0 and s-linearity
invariants, the merged-weight identity W_eff of Section 2.2 per segment, invariance
under table reordering / segment splitting / the is_finetune flag, and central finite
differences for every gradient; for the variants, the published SplitMix64 test vector, the
p = 0 and keep-frequency checks, finite differences through the masked forward, the
zero-padding identity against per-adapter matrices of their own ranks, and central finite
differences of ``forward_ragged`` for every output of ``backward_ragged``.  No function here is
"parity unpinned".
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


class SegmentError(ValueError):
    """A segment table that the layer must refuse."""


def _f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------------------
# LoRA dropout: counter-based keep mask
# --------------------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def splitmix64_output(seed: int, index: int) -> int:
    """Output number ``index`` (1-based) of the SplitMix64 stream whose state starts at ``seed``."""
    z = (seed + index * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def dropout_threshold(p: float) -> int:
    return int(round(p * 65536.0))


def dropout_keep(seed: int, n_rows: int, d_in: int, p: float) -> np.ndarray:
    """keep[m, k] (bool) for save-order rows m < n_rows and input columns k < d_in."""
    thr = dropout_threshold(p)
    keep = np.ones((n_rows, d_in), dtype=bool)
    for m in range(n_rows):
        for k4 in range((d_in + 3) // 4):
            z = splitmix64_output(seed, ((m << 32) | k4) + 1)
            for j in range(4):
                k = 4 * k4 + j
                if k < d_in:
                    keep[m, k] = ((z >> (16 * j)) & 0xFFFF) >= thr
    return keep


def dropout_keep_vectorised(seed: int, n_rows: int, d_in: int, p: float) -> np.ndarray:
    """Same mask as :func:`dropout_keep`, the generator written with numpy uint64 arrays (for the
    large cases, where the Python loops would take minutes); pinned against the loop version."""
    thr = dropout_threshold(p)
    k4 = (d_in + 3) // 4
    with np.errstate(over="ignore"):
        c = (np.arange(n_rows, dtype=np.uint64)[:, None] << np.uint64(32)) | np.arange(k4, dtype=np.uint64)[None, :]
        z = np.uint64(seed) + (c + np.uint64(1)) * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    fields = np.stack([(z >> np.uint64(16 * j)) & np.uint64(0xFFFF) for j in range(4)], axis=-1)
    return (fields.reshape(n_rows, 4 * k4)[:, :d_in] >= np.uint64(thr))


# --------------------------------------------------------------------------------------
# segment table -> per-row routing and save-buffer offsets
# --------------------------------------------------------------------------------------
def route(segments, n_rows: int, n_adapters: int):
    """Resolve a segment table.

    Returns ``(row_adapter, ft_segments, ft_rows, ft_adapters)`` where

    * ``row_adapter[t]`` is the adapter of row t, or -1 (rows outside every segment and
      segments with adapter -1 use the base weight only);
    * ``ft_segments`` lists, in table order, ``(row_start, row_len, adapter, save_offset)``
      for the fine-tuning segments; ``save_offset`` is the exclusive prefix sum of the
      fine-tuning lengths before it, i.e. where its rows land in the activation buffer;
    * ``ft_rows`` is the total number of fine-tuning rows;
    * ``ft_adapters`` lists the distinct fine-tuning adapters in order of first
      appearance; gradient slot g belongs to ``ft_adapters[g]``.

    Refused tables: negative length, rows outside [0, n_rows), two segments sharing a
    row, adapter id outside [-1, n_adapters), a fine-tuning segment without an adapter.
    Zero-length segments are legal and do nothing.
    """
    row_adapter = np.full(n_rows, -1, dtype=np.int64)
    taken = np.zeros(n_rows, dtype=bool)
    ft_segments: List[Tuple[int, int, int, int]] = []
    ft_adapters: List[int] = []
    off = 0
    for seg in np.asarray(segments, dtype=np.int64).reshape(-1, 4):
        start, length, adapter, is_ft = (int(v) for v in seg)
        if length < 0 or start < 0 or start + length > n_rows:
            raise SegmentError(f"segment ({start},{length}) outside [0,{n_rows})")
        if adapter < -1 or adapter >= n_adapters:
            raise SegmentError(f"adapter id {adapter} outside [-1,{n_adapters})")
        if is_ft and adapter < 0:
            raise SegmentError("fine-tuning segment needs an adapter")
        if taken[start:start + length].any():
            raise SegmentError(f"segment ({start},{length}) overlaps another")
        taken[start:start + length] = True
        row_adapter[start:start + length] = adapter
        if is_ft:
            ft_segments.append((start, length, adapter, off))
            off += length
            if adapter not in ft_adapters:
                ft_adapters.append(adapter)
    return row_adapter, ft_segments, off, ft_adapters


# --------------------------------------------------------------------------------------
# forward
# --------------------------------------------------------------------------------------
def forward(X, W, A_all, B_all, scale, segments, save_row_base: int = 0,
            save_capacity_rows: Optional[int] = None, dropout: Optional[Tuple[float, int]] = None) -> Dict[str, np.ndarray]:
    """Y = X W + s_a (X A_a^T) B_a per row, plus the activation save for fine-tuning rows.

    Shapes: X [T, d_in], W [d_in, d_out], A_all [n, r, d_in], B_all [n, r, d_out],
    scale [n].  Returns a dict with ``Y`` [T, d_out], ``U`` [T, r] (zero for rows without
    an adapter), ``x_save`` [capacity, d_in] and ``u_save`` [capacity, r] (rows outside
    [base, base + ft_rows) left at zero), ``ft_rows``, ``ft_adapters``.

    Save order (Section 3.2: activations are appended to a buffer of limited capacity that
    the backward later consumes): fine-tuning segments in table order, rows in order inside
    each; a batch that does not fit the remaining capacity is refused.

    ``dropout`` = (p, seed) switches LoRA dropout on for the fine-tuning rows (see the module
    header); row m of the mask is the row's place in this batch's save order (without the base).
    """
    X, W, A_all, B_all, scale = _f64(X), _f64(W), _f64(A_all), _f64(B_all), _f64(scale)
    T, d_in = X.shape
    d_out = W.shape[1]
    n, r = A_all.shape[0], A_all.shape[1]
    row_adapter, ft_segments, ft_rows, ft_adapters = route(segments, T, n)
    cap = save_row_base + ft_rows if save_capacity_rows is None else save_capacity_rows
    if save_row_base < 0 or save_row_base + ft_rows > cap:
        raise SegmentError("fine-tuning rows exceed the activation buffer capacity")

    save_place = np.full(T, -1, dtype=np.int64)  # place of a fine-tuning row in this batch's save order
    for start, length, _adapter, off in ft_segments:
        save_place[start:start + length] = off + np.arange(length)
    keep = dropout_keep(dropout[1], ft_rows, d_in, dropout[0]) if dropout is not None else None

    Y = X @ W                                   # the shared base pass
    U = np.zeros((T, r))
    for t in range(T):
        a = row_adapter[t]
        if a < 0:
            continue
        x_lora = X[t]
        if keep is not None and save_place[t] >= 0:
            x_lora = X[t] * keep[save_place[t]] / (1.0 - dropout[0])   # dropout on the branch input
        U[t] = A_all[a] @ x_lora                # shrink:  u = x A_a^T
        Y[t] += scale[a] * (U[t] @ B_all[a])    # expand:  y += s u B_a

    x_save = np.zeros((cap, d_in))
    u_save = np.zeros((cap, r))
    for start, length, _adapter, off in ft_segments:
        for i in range(length):
            m = save_row_base + off + i
            x_save[m] = X[start + i]
            u_save[m] = U[start + i]
    return {"Y": Y, "U": U, "x_save": x_save, "u_save": u_save, "ft_rows": ft_rows,
            "ft_adapters": ft_adapters, "row_adapter": row_adapter}


def forward_ragged(X, W, A_list, B_list, scale, segments) -> np.ndarray:
    """Y when adapter a has its own rank: ``A_list[a]`` [r_a, d_in], ``B_list[a]`` [r_a, d_out]."""
    X, W, scale = _f64(X), _f64(W), _f64(scale)
    row_adapter, _, _, _ = route(segments, X.shape[0], len(A_list))
    Y = X @ W
    for t in range(X.shape[0]):
        a = row_adapter[t]
        if a >= 0:
            Y[t] += scale[a] * ((_f64(A_list[a]) @ X[t]) @ _f64(B_list[a]))
    return Y


def pad_adapters(A_list, B_list, r: int):
    """Stack per-adapter matrices of different ranks into [n, r, d] arrays with zero rows."""
    n = len(A_list)
    A_all = np.zeros((n, r, np.asarray(A_list[0]).shape[1]))
    B_all = np.zeros((n, r, np.asarray(B_list[0]).shape[1]))
    for a in range(n):
        ra = np.asarray(A_list[a]).shape[0]
        A_all[a, :ra] = A_list[a]
        B_all[a, :ra] = B_list[a]
    return A_all, B_all


def forward_rows(X, W, A_all, B_all, scale, segments, rows: Sequence[int]) -> np.ndarray:
    """Y for the listed rows only (same definition; lets large cases be sampled)."""
    X, W, A_all, B_all, scale = _f64(X), _f64(W), _f64(A_all), _f64(B_all), _f64(scale)
    row_adapter, _, _, _ = route(segments, X.shape[0], A_all.shape[0])
    rows = np.asarray(rows, dtype=np.int64)
    Y = X[rows] @ W
    for i, t in enumerate(rows):
        a = row_adapter[t]
        if a >= 0:
            Y[i] += scale[a] * ((A_all[a] @ X[t]) @ B_all[a])
    return Y


# --------------------------------------------------------------------------------------
# backward (fine-tuning rows only, in save-buffer order)
# --------------------------------------------------------------------------------------
def backward(dY, W, A_all, B_all, scale, segments, x_save, u_save, n_rows: Optional[int] = None,
             dA_init=None, dB_init=None, dropout: Optional[Tuple[float, int]] = None) -> Dict[str, np.ndarray]:
    """LoRA gradients and input gradient for the fine-tuning rows.

    ``dY`` [ft_rows, d_out], ``x_save`` [ft_rows, d_in] and ``u_save`` [ft_rows, r] are in
    save order (row m of each belongs together).  ``segments`` is the same table the forward
    saw; only its fine-tuning segments matter, through their save offsets and adapters.
    Returns ``dA`` [n_slots, r, d_in], ``dB`` [n_slots, r, d_out] (slot g = g-th distinct
    fine-tuning adapter in table order; several segments on one adapter add up), ``dX``
    [ft_rows, d_in] and ``V`` [ft_rows, r].  ``dA_init`` / ``dB_init`` are added to
    (gradient accumulation across backward batches).
    """
    dY, W, A_all, B_all, scale = _f64(dY), _f64(W), _f64(A_all), _f64(B_all), _f64(scale)
    x_save, u_save = _f64(x_save), _f64(u_save)
    n, r, d_in = A_all.shape
    d_out = B_all.shape[2]
    if n_rows is None:
        seg = np.asarray(segments, dtype=np.int64).reshape(-1, 4)
        n_rows = int((seg[:, 0] + seg[:, 1]).max()) if len(seg) else 0
    _, ft_segments, ft_rows, ft_adapters = route(segments, n_rows, n)
    if dY.shape[0] != ft_rows:
        raise SegmentError("dY must have one row per fine-tuning row")

    dA = np.zeros((len(ft_adapters), r, d_in)) if dA_init is None else _f64(dA_init).copy()
    dB = np.zeros((len(ft_adapters), r, d_out)) if dB_init is None else _f64(dB_init).copy()
    dX = np.zeros((ft_rows, d_in))
    V = np.zeros((ft_rows, r))
    keep = dropout_keep(dropout[1], ft_rows, d_in, dropout[0]) if dropout is not None else None
    for _start, length, a, off in ft_segments:
        g = ft_adapters.index(a)
        s = scale[a]
        for m in range(off, off + length):
            V[m] = s * (B_all[a] @ dY[m])                  # v = s dy B_a^T
            dB[g] += s * np.outer(u_save[m], dY[m])        # dB_a += s u^T dy
            if keep is None:
                dA[g] += np.outer(V[m], x_save[m])         # dA_a += v^T x
                dX[m] = W @ dY[m] + V[m] @ A_all[a]        # dx = dy W^T + v A_a
            else:
                k = keep[m] / (1.0 - dropout[0])
                dA[g] += np.outer(V[m], x_save[m] * k)     # the branch saw x * k
                dX[m] = W @ dY[m] + (V[m] @ A_all[a]) * k
    return {"dA": dA, "dB": dB, "dX": dX, "V": V, "ft_adapters": ft_adapters}


def backward_ragged(dY, W, A_list, B_list, scale, segments, x_save, n_rows: int):
    """Gradients when adapter a has its own rank r_a (Section 2.2: many adapters share one base model; nothing makes
    them share a rank):
    the same chain rule as ``backward`` with each adapter's own matrices, nothing padded.  ``u`` is recomputed
    from the saved input (u = A_a x), since saved rows of different adapters would have different widths.
    Returns ``dA`` and ``dB`` as lists (slot g: [r_a, d_in] and [r_a, d_out]), ``dX`` [ft_rows, d_in] and
    ``ft_adapters``."""
    dY, W, scale, x_save = _f64(dY), _f64(W), _f64(scale), _f64(x_save)
    _, ft_segments, ft_rows, ft_adapters = route(segments, n_rows, len(A_list))
    if dY.shape[0] != ft_rows:
        raise SegmentError("dY must have one row per fine-tuning row")
    dA = [np.zeros_like(_f64(A_list[a])) for a in ft_adapters]
    dB = [np.zeros_like(_f64(B_list[a])) for a in ft_adapters]
    dX = np.zeros((ft_rows, W.shape[0]))
    for _start, length, a, off in ft_segments:
        g = ft_adapters.index(a)
        A, B, s = _f64(A_list[a]), _f64(B_list[a]), scale[a]
        for m in range(off, off + length):
            u = A @ x_save[m]                              # u = x A_a^T
            v = s * (B @ dY[m])                            # v = s dy B_a^T
            dB[g] += s * np.outer(u, dY[m])
            dA[g] += np.outer(v, x_save[m])
            dX[m] = W @ dY[m] + v @ A
    return {"dA": dA, "dB": dB, "dX": dX, "ft_adapters": ft_adapters}


def backward_blocked(dY, W, A_all, B_all, scale, segments, x_save, u_save,
                     n_rows: Optional[int] = None, dropout: Optional[Tuple[float, int]] = None) -> Dict[str, np.ndarray]:
    """Same result as :func:`backward`, one library matrix product per segment instead of one
    row at a time (the sums over a segment's rows are exactly the matrix products
    U^T dY, V^T X, dY W^T); used where the row loop would take minutes."""
    dY, W, A_all, B_all, scale = _f64(dY), _f64(W), _f64(A_all), _f64(B_all), _f64(scale)
    x_save, u_save = _f64(x_save), _f64(u_save)
    n, r, d_in = A_all.shape
    d_out = B_all.shape[2]
    if n_rows is None:
        seg = np.asarray(segments, dtype=np.int64).reshape(-1, 4)
        n_rows = int((seg[:, 0] + seg[:, 1]).max()) if len(seg) else 0
    _, ft_segments, ft_rows, ft_adapters = route(segments, n_rows, n)
    dA = np.zeros((len(ft_adapters), r, d_in))
    dB = np.zeros((len(ft_adapters), r, d_out))
    dX = np.zeros((ft_rows, d_in))
    V = np.zeros((ft_rows, r))
    k = np.ones((ft_rows, d_in))
    if dropout is not None:
        k = dropout_keep_vectorised(dropout[1], ft_rows, d_in, dropout[0]) / (1.0 - dropout[0])
    for _start, length, a, off in ft_segments:
        g = ft_adapters.index(a)
        sl = slice(off, off + length)
        V[sl] = scale[a] * (dY[sl] @ B_all[a].T)
        dB[g] += scale[a] * (u_save[sl].T @ dY[sl])
        dA[g] += V[sl].T @ (x_save[sl] * k[sl])
        dX[sl] = dY[sl] @ W.T + (V[sl] @ A_all[a]) * k[sl]
    return {"dA": dA, "dB": dB, "dX": dX, "V": V, "ft_adapters": ft_adapters}


def forward_blocked(X, W, A_all, B_all, scale, segments, dropout: Optional[Tuple[float, int]] = None) -> Dict[str, np.ndarray]:
    """Same result as :func:`forward` (without the save buffers), one library product per
    segment instead of one row at a time; used for the timed CPU baseline and large cases."""
    X, W, A_all, B_all, scale = _f64(X), _f64(W), _f64(A_all), _f64(B_all), _f64(scale)
    T = X.shape[0]
    n, r = A_all.shape[0], A_all.shape[1]
    _ra, ft_segments, ft_rows, ft_adapters = route(segments, T, n)
    Y = X @ W
    U = np.zeros((T, r))
    keep = dropout_keep_vectorised(dropout[1], ft_rows, X.shape[1], dropout[0]) if dropout is not None else None
    ft_off = {(st, ln): off for st, ln, _a, off in ft_segments}
    for seg in np.asarray(segments, dtype=np.int64).reshape(-1, 4):
        start, length, a, is_ft = (int(v) for v in seg)
        if a < 0 or length == 0:
            continue
        sl = slice(start, start + length)
        x_lora = X[sl]
        if keep is not None and is_ft:
            off = ft_off[(start, length)]
            x_lora = X[sl] * keep[off:off + length] / (1.0 - dropout[0])
        U[sl] = x_lora @ A_all[a].T
        Y[sl] += scale[a] * (U[sl] @ B_all[a])
    x_save = np.zeros((ft_rows, X.shape[1]))
    u_save = np.zeros((ft_rows, r))
    for start, length, _a, off in ft_segments:
        x_save[off:off + length] = X[start:start + length]
        u_save[off:off + length] = U[start:start + length]
    return {"Y": Y, "U": U, "x_save": x_save, "u_save": u_save, "ft_rows": ft_rows,
            "ft_adapters": ft_adapters}
