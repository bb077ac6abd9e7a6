"""Pins for the CPU oracle: it is checked against things other than itself.

* brute force, element by element, in pure Python on tiny shapes (written here independently);
* a worked example computed by hand (tests/golden/worked_example.txt);
* invariants the mathematics fixes: B = 0, linearity in s, the merged weight
  W_eff = W + B A of Section 2.2 per segment, table reordering / segment splitting, the
  is_finetune flag not changing Y (Section 3.2: the fine-tuning forward is the inference forward);
* central finite differences for every gradient (the loss <dY, Y> is linear in A, in B and
  in X, so the differences are exact up to round-off);
* the activation-memory arithmetic the paper prints (Section 3.2: N_L d p bytes per token).
"""
import itertools
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from oracle import mlora_oracle as orc  # noqa: E402
from paper_2607_28848_b200 import synth  # noqa: E402


# ---------------------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------------------
def small_problem(seed=0, d_in=5, d_out=7, r=2, n=3, T=9, segs=None):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((T, d_in))
    W = rng.standard_normal((d_in, d_out))
    A = rng.standard_normal((n, r, d_in))
    B = rng.standard_normal((n, r, d_out))
    s = rng.uniform(0.5, 3.0, n)
    if segs is None:
        segs = [(0, 2, 1, 0), (2, 3, 0, 1), (5, 1, 2, 0), (7, 2, 1, 1)]   # row 6 uncovered
    return X, W, A, B, s, np.asarray(segs, dtype=np.int32)


def brute_forward(X, W, A, B, s, segs):
    """y[t][j] = sum_k x[t][k] w[k][j] + s_a sum_q (sum_k x[t][k] a[q][k]) b[q][j], scalar loops."""
    T, d_in = len(X), len(X[0])
    d_out = len(W[0])
    r = len(A[0])
    adapter = [-1] * T
    for st, ln, ad, _ in segs:
        for t in range(st, st + ln):
            adapter[t] = ad
    Y = [[0.0] * d_out for _ in range(T)]
    U = [[0.0] * r for _ in range(T)]
    for t in range(T):
        for j in range(d_out):
            acc = 0.0
            for k in range(d_in):
                acc += X[t][k] * W[k][j]
            Y[t][j] = acc
        a = adapter[t]
        if a < 0:
            continue
        for q in range(r):
            acc = 0.0
            for k in range(d_in):
                acc += X[t][k] * A[a][q][k]
            U[t][q] = acc
        for j in range(d_out):
            acc = 0.0
            for q in range(r):
                acc += U[t][q] * B[a][q][j]
            Y[t][j] += s[a] * acc
    return Y, U, adapter


def brute_backward(dY, W, A, B, s, ft_rows_adapters, xs, us, slots):
    """Scalar-loop chain rule; ft_rows_adapters[m] = adapter of saved row m."""
    M = len(dY)
    d_out = len(dY[0])
    d_in = len(xs[0])
    r = len(us[0])
    dA = [[[0.0] * d_in for _ in range(r)] for _ in slots]
    dB = [[[0.0] * d_out for _ in range(r)] for _ in slots]
    dX = [[0.0] * d_in for _ in range(M)]
    for m in range(M):
        a = ft_rows_adapters[m]
        g = slots.index(a)
        v = [0.0] * r
        for q in range(r):
            acc = 0.0
            for j in range(d_out):
                acc += dY[m][j] * B[a][q][j]
            v[q] = s[a] * acc
        for q in range(r):
            for j in range(d_out):
                dB[g][q][j] += s[a] * us[m][q] * dY[m][j]
            for k in range(d_in):
                dA[g][q][k] += v[q] * xs[m][k]
        for k in range(d_in):
            acc = 0.0
            for j in range(d_out):
                acc += dY[m][j] * W[k][j]
            for q in range(r):
                acc += v[q] * A[a][q][k]
            dX[m][k] = acc
    return dA, dB, dX


FORWARDS = [orc.forward, orc.forward_blocked]
BACKWARDS = [orc.backward, orc.backward_blocked]


# ---------------------------------------------------------------------------------------
# worked example (hand-computed)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("fwd,bwd", list(zip(FORWARDS, BACKWARDS)))
def test_worked_example(golden_example, fwd, bwd):
    g = golden_example
    A = np.stack([g["A0"], g["A1"]])
    B = np.stack([g["B0"], g["B1"]])
    s = g["scale"][0]
    segs = g["segments"].astype(np.int32)
    out = fwd(g["X"], g["W"], A, B, s, segs)
    assert np.array_equal(out["Y"], g["Y"])
    assert np.array_equal(out["U"], g["U"])
    assert np.array_equal(out["x_save"], g["x_save"])
    assert np.array_equal(out["u_save"], g["u_save"])
    assert out["ft_rows"] == 2 and out["ft_adapters"] == [1]
    back = bwd(g["dY"], g["W"], A, B, s, segs, out["x_save"], out["u_save"], n_rows=3)
    assert np.array_equal(back["V"], g["V"])
    assert np.array_equal(back["dB"][0], g["dB"])
    assert np.array_equal(back["dA"][0], g["dA"])
    assert np.array_equal(back["dX"], g["dX"])


# ---------------------------------------------------------------------------------------
# brute force
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("fwd,bwd", list(zip(FORWARDS, BACKWARDS)))
def test_brute_force_tiny(seed, fwd, bwd):
    X, W, A, B, s, segs = small_problem(seed)
    out = fwd(X, W, A, B, s, segs)
    Yb, Ub, adapter = brute_forward(X.tolist(), W.tolist(), A.tolist(), B.tolist(), s.tolist(), segs.tolist())
    np.testing.assert_allclose(out["Y"], np.asarray(Yb), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(out["U"], np.asarray(Ub), rtol=1e-13, atol=1e-13)
    # save order: fine-tune segments in table order -> rows 2,3,4 then 7,8
    ft_rows = [2, 3, 4, 7, 8]
    assert out["ft_rows"] == 5
    assert np.array_equal(out["x_save"], X[ft_rows])
    np.testing.assert_allclose(out["u_save"], np.asarray(Ub)[ft_rows], rtol=1e-13, atol=1e-13)
    assert out["ft_adapters"] == [0, 1]

    rng = np.random.default_rng(100 + seed)
    dY = rng.standard_normal((5, W.shape[1]))
    back = bwd(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X))
    dAb, dBb, dXb = brute_backward(dY.tolist(), W.tolist(), A.tolist(), B.tolist(), s.tolist(),
                                   [adapter[t] for t in ft_rows], X[ft_rows].tolist(),
                                   np.asarray(Ub)[ft_rows].tolist(), [0, 1])
    np.testing.assert_allclose(back["dA"], np.asarray(dAb), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(back["dB"], np.asarray(dBb), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(back["dX"], np.asarray(dXb), rtol=1e-12, atol=1e-12)


def test_blocked_variants_agree_with_rowwise():
    w = synth.random_workload(3, 24, 40, 4, 5, 150, dtype="f32", max_seg=30)
    t = synth.make_tensors(w)
    a = orc.forward(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)
    b = orc.forward_blocked(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments)
    np.testing.assert_allclose(a["Y"], b["Y"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(a["U"], b["U"], rtol=1e-12, atol=1e-12)
    assert np.array_equal(a["x_save"], b["x_save"])
    np.testing.assert_allclose(a["u_save"], b["u_save"], rtol=1e-12, atol=1e-12)
    ga = orc.backward(t["dY"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments,
                      a["x_save"], a["u_save"], n_rows=w.n_rows)
    gb = orc.backward_blocked(t["dY"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments,
                              a["x_save"], a["u_save"], n_rows=w.n_rows)
    for k in ("dA", "dB", "dX", "V"):
        np.testing.assert_allclose(ga[k], gb[k], rtol=1e-11, atol=1e-11)
    rows = [0, 7, 33, 149]
    np.testing.assert_allclose(
        orc.forward_rows(t["X"], t["W"], t["A_all"], t["B_all"], t["scale"], w.segments, rows),
        a["Y"][rows], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------------------------
# forward invariants
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("fwd", FORWARDS)
def test_zero_B_gives_base_gemm_exactly(fwd):
    X, W, A, B, s, segs = small_problem(4)
    out = fwd(X, W, A, np.zeros_like(B), s, segs)
    assert np.array_equal(out["Y"], X @ W)


@pytest.mark.parametrize("fwd", FORWARDS)
def test_linearity_in_scale(fwd):
    X, W, A, B, s, segs = small_problem(5)
    n = len(s)
    y0 = fwd(X, W, A, B, np.zeros(n), segs)["Y"]
    y1 = fwd(X, W, A, B, np.ones(n), segs)["Y"]
    ys = fwd(X, W, A, B, s, segs)["Y"]
    row_adapter, _, _, _ = orc.route(segs, len(X), n)
    srow = np.where(row_adapter >= 0, s[np.maximum(row_adapter, 0)], 0.0)[:, None]
    np.testing.assert_allclose(ys - y0, srow * (y1 - y0), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("fwd", FORWARDS)
def test_merged_weight_per_segment(fwd):
    """Section 2.2: a segment's rows see the effective weight W + s A_a^T B_a."""
    X, W, A, B, s, segs = small_problem(6)
    Y = fwd(X, W, A, B, s, segs)["Y"]
    covered = np.zeros(len(X), dtype=bool)
    for st, ln, ad, _ in segs.tolist():
        w_eff = W + s[ad] * np.einsum("qk,qj->kj", A[ad], B[ad])
        np.testing.assert_allclose(Y[st:st + ln], X[st:st + ln] @ w_eff, rtol=1e-12, atol=1e-12)
        covered[st:st + ln] = True
    assert np.array_equal(Y[~covered], (X @ W)[~covered])          # uncovered rows: base only


@pytest.mark.parametrize("fwd", FORWARDS)
def test_adapter_minus_one_is_base_only(fwd):
    X, W, A, B, s, _ = small_problem(7)
    segs = np.asarray([(0, 4, -1, 0), (4, 5, 2, 0)], dtype=np.int32)
    Y = fwd(X, W, A, B, s, segs)["Y"]
    assert np.array_equal(Y[:4], (X @ W)[:4])
    assert not np.allclose(Y[4:], (X @ W)[4:])


@pytest.mark.parametrize("fwd", FORWARDS)
def test_finetune_flag_does_not_change_Y(fwd):
    X, W, A, B, s, segs = small_problem(8)
    flipped = segs.copy()
    flipped[:, 3] = 1 - flipped[:, 3]
    assert np.array_equal(fwd(X, W, A, B, s, segs)["Y"], fwd(X, W, A, B, s, flipped)["Y"])


@pytest.mark.parametrize("fwd", FORWARDS)
def test_table_reorder_and_split(fwd):
    X, W, A, B, s, segs = small_problem(9)
    base = fwd(X, W, A, B, s, segs)
    # split the first fine-tune segment (rows 2..4) in two: same Y, same save order
    split = np.asarray([(0, 2, 1, 0), (2, 1, 0, 1), (3, 2, 0, 1), (5, 1, 2, 0), (7, 2, 1, 1)], dtype=np.int32)
    o2 = fwd(X, W, A, B, s, split)
    np.testing.assert_allclose(base["Y"], o2["Y"], rtol=1e-13, atol=1e-13)
    assert np.array_equal(base["x_save"], o2["x_save"])
    # reorder the table: Y unchanged, save order follows the table
    perm = segs[[3, 0, 2, 1]]
    o3 = fwd(X, W, A, B, s, perm)
    np.testing.assert_allclose(base["Y"], o3["Y"], rtol=1e-13, atol=1e-13)
    assert np.array_equal(o3["x_save"], X[[7, 8, 2, 3, 4]])
    assert o3["ft_adapters"] == [1, 0]


def test_row_permutation_consistency():
    X, W, A, B, s, _ = small_problem(10, T=8)
    segs = np.asarray([(0, 3, 0, 0), (3, 5, 2, 0)], dtype=np.int32)
    Y = orc.forward(X, W, A, B, s, segs)["Y"]
    # move the second segment in front of the first
    Xp = np.concatenate([X[3:], X[:3]])
    segp = np.asarray([(5, 3, 0, 0), (0, 5, 2, 0)], dtype=np.int32)
    Yp = orc.forward(Xp, W, A, B, s, segp)["Y"]
    np.testing.assert_allclose(Yp, np.concatenate([Y[3:], Y[:3]]), rtol=1e-13, atol=1e-13)


def test_save_base_and_capacity():
    X, W, A, B, s, segs = small_problem(11)
    out = orc.forward(X, W, A, B, s, segs, save_row_base=3, save_capacity_rows=8)
    assert np.array_equal(out["x_save"][3:8], X[[2, 3, 4, 7, 8]])
    assert not out["x_save"][:3].any()
    with pytest.raises(orc.SegmentError):
        orc.forward(X, W, A, B, s, segs, save_row_base=4, save_capacity_rows=8)


# ---------------------------------------------------------------------------------------
# routing / error paths
# ---------------------------------------------------------------------------------------
def test_route_offsets_hand_listed():
    segs = [(10, 4, 2, 1), (0, 3, 1, 0), (3, 0, 0, 1), (20, 5, 0, 1), (4, 2, 2, 1)]
    row_adapter, ft, ft_rows, slots = orc.route(segs, 30, 3)
    assert ft == [(10, 4, 2, 0), (3, 0, 0, 4), (20, 5, 0, 4), (4, 2, 2, 9)]
    assert ft_rows == 11
    assert slots == [2, 0]
    assert row_adapter[:7].tolist() == [1, 1, 1, -1, 2, 2, -1]


@pytest.mark.parametrize("bad", [
    [(0, 5, 0, 0), (4, 2, 1, 0)],        # overlap
    [(28, 5, 0, 0)],                     # out of range
    [(-1, 2, 0, 0)],                     # negative start
    [(0, -2, 0, 0)],                     # negative length
    [(0, 2, 3, 0)],                      # adapter id too large
    [(0, 2, -2, 0)],                     # adapter id below -1
    [(0, 2, -1, 1)],                     # fine-tune without adapter
])
def test_route_refuses(bad):
    with pytest.raises(orc.SegmentError):
        orc.route(bad, 30, 3)


# ---------------------------------------------------------------------------------------
# gradients
# ---------------------------------------------------------------------------------------
def _loss(X, W, A, B, s, segs, dY):
    out = orc.forward(X, W, A, B, s, segs)
    _, ft, _, _ = orc.route(segs, len(X), len(s))
    tot = 0.0
    for st, ln, _a, off in ft:
        tot += float(np.sum(dY[off:off + ln] * out["Y"][st:st + ln]))
    return tot


@pytest.mark.parametrize("bwd", BACKWARDS)
def test_finite_differences(bwd):
    X, W, A, B, s, segs = small_problem(12)
    rng = np.random.default_rng(5)
    out = orc.forward(X, W, A, B, s, segs)
    dY = rng.standard_normal((out["ft_rows"], W.shape[1]))
    back = bwd(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X))
    slots = back["ft_adapters"]
    h = 0.5
    for g, a in enumerate(slots):
        for q, k in itertools.product(range(A.shape[1]), range(A.shape[2])):
            Ap, Am = A.copy(), A.copy()
            Ap[a, q, k] += h
            Am[a, q, k] -= h
            fd = (_loss(X, W, Ap, B, s, segs, dY) - _loss(X, W, Am, B, s, segs, dY)) / (2 * h)
            assert abs(fd - back["dA"][g, q, k]) <= 1e-9 * (1 + abs(fd))
        for q, j in itertools.product(range(B.shape[1]), range(B.shape[2])):
            Bp, Bm = B.copy(), B.copy()
            Bp[a, q, j] += h
            Bm[a, q, j] -= h
            fd = (_loss(X, W, A, Bp, s, segs, dY) - _loss(X, W, A, Bm, s, segs, dY)) / (2 * h)
            assert abs(fd - back["dB"][g, q, j]) <= 1e-9 * (1 + abs(fd))
    _, ft, _, _ = orc.route(segs, len(X), len(s))
    for st, ln, _a, off in ft:
        for i, k in itertools.product(range(ln), range(X.shape[1])):
            Xp, Xm = X.copy(), X.copy()
            Xp[st + i, k] += h
            Xm[st + i, k] -= h
            fd = (_loss(Xp, W, A, B, s, segs, dY) - _loss(Xm, W, A, B, s, segs, dY)) / (2 * h)
            assert abs(fd - back["dX"][off + i, k]) <= 1e-9 * (1 + abs(fd))


@pytest.mark.parametrize("bwd", BACKWARDS)
def test_dX_is_merged_weight_transpose(bwd):
    X, W, A, B, s, segs = small_problem(13)
    rng = np.random.default_rng(6)
    out = orc.forward(X, W, A, B, s, segs)
    dY = rng.standard_normal((out["ft_rows"], W.shape[1]))
    back = bwd(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X))
    _, ft, _, _ = orc.route(segs, len(X), len(s))
    for _st, ln, a, off in ft:
        w_eff = W + s[a] * np.einsum("qk,qj->kj", A[a], B[a])
        np.testing.assert_allclose(back["dX"][off:off + ln], dY[off:off + ln] @ w_eff.T, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("bwd", BACKWARDS)
def test_gradient_structure(bwd):
    X, W, A, B, s, segs = small_problem(14)
    rng = np.random.default_rng(7)
    out = orc.forward(X, W, A, B, s, segs)
    dY = rng.standard_normal((out["ft_rows"], W.shape[1]))
    full = bwd(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X))
    # two fine-tune segments on one adapter: gradient = sum of the two single-segment gradients
    same = np.asarray([(2, 3, 1, 1), (7, 2, 1, 1)], dtype=np.int32)
    o = orc.forward(X, W, A, B, s, same)
    both = bwd(dY, W, A, B, s, same, o["x_save"], o["u_save"], n_rows=len(X))
    s1 = np.asarray([(2, 3, 1, 1)], dtype=np.int32)
    s2 = np.asarray([(7, 2, 1, 1)], dtype=np.int32)
    o1, o2 = orc.forward(X, W, A, B, s, s1), orc.forward(X, W, A, B, s, s2)
    g1 = bwd(dY[:3], W, A, B, s, s1, o1["x_save"], o1["u_save"], n_rows=len(X))
    g2 = bwd(dY[3:], W, A, B, s, s2, o2["x_save"], o2["u_save"], n_rows=len(X))
    np.testing.assert_allclose(both["dA"], g1["dA"] + g2["dA"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(both["dB"], g1["dB"] + g2["dB"], rtol=1e-12, atol=1e-12)
    # gradients do not depend on the inference rows of the batch
    only_ft = segs[segs[:, 3] != 0]
    o_ft = orc.forward(X, W, A, B, s, only_ft)
    g_ft = bwd(dY, W, A, B, s, only_ft, o_ft["x_save"], o_ft["u_save"], n_rows=len(X))
    for k in ("dA", "dB", "dX"):
        np.testing.assert_allclose(full[k], g_ft[k], rtol=1e-13, atol=1e-13)
    # dA, dB and the adapter part of dX are linear in s
    s2x = 2.0 * s
    o2x = orc.forward(X, W, A, B, s2x, segs)
    g2x = bwd(dY, W, A, B, s2x, segs, o2x["x_save"], o2x["u_save"], n_rows=len(X))
    np.testing.assert_allclose(g2x["dA"], 2 * full["dA"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g2x["dB"], 2 * full["dB"], rtol=1e-12, atol=1e-12)
    base_dx = dY @ W.T
    np.testing.assert_allclose(g2x["dX"] - base_dx, 2 * (full["dX"] - base_dx), rtol=1e-11, atol=1e-11)


def test_accumulate_adds():
    X, W, A, B, s, segs = small_problem(15)
    rng = np.random.default_rng(8)
    out = orc.forward(X, W, A, B, s, segs)
    dY = rng.standard_normal((out["ft_rows"], W.shape[1]))
    g = orc.backward(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X))
    g2 = orc.backward(dY, W, A, B, s, segs, out["x_save"], out["u_save"], n_rows=len(X),
                      dA_init=g["dA"], dB_init=g["dB"])
    np.testing.assert_allclose(g2["dA"], 2 * g["dA"], rtol=1e-13)
    np.testing.assert_allclose(g2["dB"], 2 * g["dB"], rtol=1e-13)


# ---------------------------------------------------------------------------------------
# exact-arithmetic routing probe: every value is a small integer, so the result is exact
# ---------------------------------------------------------------------------------------
def test_integer_probe_is_exact():
    from probes import integer_probe
    p = integer_probe(n_rows=40, d_in=16, d_out=16, rank=8, n_adapters=4, seed=3)
    out = orc.forward(p["X"], p["W"], p["A_all"], p["B_all"], p["scale"], p["segments"])
    assert np.array_equal(out["Y"], np.round(out["Y"]))
    assert np.abs(out["Y"]).max() < 2 ** 8          # exactly representable in bf16 as well
    Yb, _, _ = brute_forward(p["X"].tolist(), p["W"].tolist(), p["A_all"].tolist(), p["B_all"].tolist(),
                             p["scale"].tolist(), p["segments"].tolist())
    assert np.array_equal(out["Y"], np.asarray(Yb))


# ---------------------------------------------------------------------------------------
# numbers the paper prints
# ---------------------------------------------------------------------------------------
def test_activation_bytes_per_token():
    """Section 3.2: saving only each layer's input costs N_L * d * p bytes per token,
    about 0.25 MB for N_L = 32, d = 4096, 16-bit activations."""
    n_layers, d, p = 32, 4096, 2
    per_layer = d * p                         # one saved X row of a d-wide projection
    assert per_layer == 8192
    assert n_layers * per_layer == 262144     # 0.25 MiB
    w = synth.cfg3_layer_set(projections=["q"])[0]
    assert w.d_in * w.elem_bytes == per_layer


def test_lora_scale_constant():
    """Section 5: r = 16, alpha = 32, hence s = alpha / r = 2 in every workload."""
    assert synth.cfg2_single_projection().lora_scale == 32 / 16
