"""Input builders for the exact-arithmetic routing probe (inputs only, no method arithmetic).

Every tensor holds small integers and every adapter matrix is a one-hot selection keyed by
the adapter id, so each output of the layer is a small integer that bf16 and fp32 represent
exactly.  A correct implementation therefore reproduces the oracle BIT FOR BIT, and a row
routed to the wrong adapter, a wrong scale or a mis-indexed save row changes an integer.
"""
import numpy as np

from paper_2607_28848_b200 import synth


def integer_probe(n_rows, d_in, d_out, rank, n_adapters, seed=0, dtype="bf16", segments=None,
                  max_seg=70, base="perm"):
    if segments is None:
        w = synth.random_workload(seed, d_in, d_out, rank, n_adapters, n_rows, dtype=dtype, max_seg=max_seg)
        segments = w.segments
    X = (synth.randint(seed, 11, n_rows * d_in, 7) - 3).reshape(n_rows, d_in).astype(np.float32)
    W = np.zeros((d_in, d_out), dtype=np.float32)
    if base == "perm":
        for k in range(d_in):                       # column (5k+1) mod d_out receives input k
            W[k, (5 * k + 1) % d_out] += 1.0 if k < d_out else 0.0
    A = np.zeros((n_adapters, rank, d_in), dtype=np.float32)
    B = np.zeros((n_adapters, rank, d_out), dtype=np.float32)
    for a in range(n_adapters):
        for q in range(rank):
            A[a, q, (7 * a + 3 * q) % d_in] = 1.0   # u[q] = x[(7a+3q) mod d_in]
            B[a, q, (11 * a + q) % d_out] = 1.0     # y[(11a+q) mod d_out] += s u[q]
    scale = np.asarray([2.0 if a % 2 == 0 else 4.0 for a in range(n_adapters)], dtype=np.float32)
    ft_rows = int(segments[segments[:, 3] != 0, 1].sum()) if len(segments) else 0
    dY = (synth.randint(seed, 12, ft_rows * d_out, 5) - 2).reshape(ft_rows, d_out).astype(np.float32)
    return {"X": X, "W": W, "A_all": A, "B_all": B, "scale": scale, "segments": segments, "dY": dY,
            "n_rows": n_rows, "d_in": d_in, "d_out": d_out, "rank": rank, "n_adapters": n_adapters,
            "dtype": dtype}
