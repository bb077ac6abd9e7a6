"""Pins for the oracle's variants: LoRA dropout (counter-based mask) and adapters of different ranks."""
import numpy as np
import pytest

from oracle import mlora_oracle as orc


def test_splitmix64_published_vector():
    # first outputs of SplitMix64 for the state 1234567 (the generator's widely published test vector)
    expect = [6457827717110365317, 3203168211198807973, 9817491932198370423, 4593380528125082431,
              16408922859458223821]
    assert [orc.splitmix64_output(1234567, i + 1) for i in range(5)] == expect


def test_keep_mask_counter_layout():
    seed, p = 99, 0.25
    keep = orc.dropout_keep(seed, 3, 10, p)
    thr = orc.dropout_threshold(p)
    assert thr == 16384
    for m, k in ((0, 0), (0, 3), (0, 4), (2, 9), (1, 7)):
        z = orc.splitmix64_output(seed, ((m << 32) | (k >> 2)) + 1)
        assert keep[m, k] == (((z >> (16 * (k & 3))) & 0xFFFF) >= thr)
    assert orc.dropout_keep(seed, 3, 10, 0.0).all()                    # p = 0 keeps everything
    assert not orc.dropout_keep(seed, 3, 10, 1.0).any()                # threshold 65536 drops everything
    assert (orc.dropout_keep(seed + 1, 3, 10, p) != keep).any()        # the seed matters
    np.testing.assert_array_equal(orc.dropout_keep(seed, 2, 10, p), keep[:2])   # rows are independent counters


def test_vectorised_mask_equals_loop_version():
    for seed, rows, d, p in ((0, 5, 17, 0.05), (2 ** 63 + 12345, 9, 64, 0.5), (7, 3, 130, 0.9)):
        np.testing.assert_array_equal(orc.dropout_keep_vectorised(seed, rows, d, p), orc.dropout_keep(seed, rows, d, p))


def test_keep_frequency():
    keep = orc.dropout_keep_vectorised(2024, 256, 4096, 0.05)
    n = keep.size
    drop = 1.0 - keep.mean()
    p_eff = orc.dropout_threshold(0.05) / 65536.0
    assert abs(drop - p_eff) < 5 * np.sqrt(p_eff * (1 - p_eff) / n)
    # per-column and per-row frequencies are unbiased too (no structure in either index)
    assert abs((1 - keep.mean(axis=0)).mean() - p_eff) < 1e-3 and (1 - keep.mean(axis=1)).max() < 0.08


def _tiny(seed=3):
    rng = np.random.default_rng(seed)
    T, d_in, d_out, r, n = 11, 12, 7, 4, 3
    X, W = rng.standard_normal((T, d_in)), rng.standard_normal((d_in, d_out))
    A, B = rng.standard_normal((n, r, d_in)), rng.standard_normal((n, r, d_out))
    scale = np.array([2.0, 0.5, 1.5])
    segs = np.array([(0, 3, 1, 0), (3, 4, 0, 1), (7, 1, 2, 0), (8, 3, 2, 1)])
    return X, W, A, B, scale, segs


def test_dropout_zero_is_the_plain_layer_and_inference_rows_never_change():
    X, W, A, B, scale, segs = _tiny()
    plain = orc.forward(X, W, A, B, scale, segs)
    same = orc.forward(X, W, A, B, scale, segs, dropout=(0.0, 5))
    np.testing.assert_allclose(same["Y"], plain["Y"], rtol=0, atol=0)
    drop = orc.forward(X, W, A, B, scale, segs, dropout=(0.5, 5))
    inf_rows = [0, 1, 2, 7]
    np.testing.assert_array_equal(drop["Y"][inf_rows], plain["Y"][inf_rows])
    assert np.abs(drop["Y"][3:7] - plain["Y"][3:7]).max() > 1e-3
    np.testing.assert_array_equal(drop["x_save"], plain["x_save"])     # the saved input is the undropped row


def test_dropout_forward_brute_force():
    X, W, A, B, scale, segs = _tiny()
    p, seed = 0.5, 11
    out = orc.forward(X, W, A, B, scale, segs, dropout=(p, seed))
    keep = orc.dropout_keep(seed, 7, X.shape[1], p)
    place = {3: 0, 4: 1, 5: 2, 6: 3, 8: 4, 9: 5, 10: 6}
    ad = {3: 0, 4: 0, 5: 0, 6: 0, 8: 2, 9: 2, 10: 2}
    for t, m in place.items():
        a = ad[t]
        for j in range(W.shape[1]):
            y = sum(X[t, k] * W[k, j] for k in range(X.shape[1]))
            for q in range(A.shape[1]):
                u = sum((X[t, k] if keep[m, k] else 0.0) / (1 - p) * A[a, q, k] for k in range(X.shape[1]))
                y += scale[a] * u * B[a, q, j]
            assert out["Y"][t, j] == pytest.approx(y, rel=1e-12, abs=1e-12)


@pytest.mark.parametrize("p", [0.0, 0.3])
def test_dropout_gradients_by_finite_differences(p):
    X, W, A, B, scale, segs = _tiny(5)
    drop = (p, 77) if p > 0 else None
    rng = np.random.default_rng(1)
    fwd = orc.forward(X, W, A, B, scale, segs, dropout=drop)
    ft_batch_rows = [3, 4, 5, 6, 8, 9, 10]                      # save order
    dY = rng.standard_normal((7, W.shape[1]))

    def loss(Xv, Av, Bv):
        return float((orc.forward(Xv, W, Av, Bv, scale, segs, dropout=drop)["Y"][ft_batch_rows] * dY).sum())
    bwd = orc.backward(dY, W, A, B, scale, segs, fwd["x_save"], fwd["u_save"], n_rows=11, dropout=drop)
    h = 1e-6
    slots = bwd["ft_adapters"]
    for g, a in enumerate(slots):
        for (q, k) in ((0, 0), (1, 5), (3, 11)):
            Ap, Am = A.copy(), A.copy(); Ap[a, q, k] += h; Am[a, q, k] -= h
            assert bwd["dA"][g, q, k] == pytest.approx((loss(X, Ap, B) - loss(X, Am, B)) / (2 * h), rel=1e-6, abs=1e-7)
        for (q, j) in ((0, 0), (2, 6)):
            Bp, Bm = B.copy(), B.copy(); Bp[a, q, j] += h; Bm[a, q, j] -= h
            assert bwd["dB"][g, q, j] == pytest.approx((loss(X, A, Bp) - loss(X, A, Bm)) / (2 * h), rel=1e-6, abs=1e-7)
    for m, t in enumerate(ft_batch_rows):
        for k in (0, 4, 11):
            Xp, Xm = X.copy(), X.copy(); Xp[t, k] += h; Xm[t, k] -= h
            assert bwd["dX"][m, k] == pytest.approx((loss(Xp, A, B) - loss(Xm, A, B)) / (2 * h), rel=1e-6, abs=1e-7)


def test_blocked_variants_agree_with_row_loops_under_dropout():
    X, W, A, B, scale, segs = _tiny(8)
    drop = (0.4, 123456789)
    f1 = orc.forward(X, W, A, B, scale, segs, dropout=drop)
    f2 = orc.forward_blocked(X, W, A, B, scale, segs, dropout=drop)
    np.testing.assert_allclose(f2["Y"], f1["Y"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f2["u_save"], f1["u_save"], rtol=1e-12, atol=1e-12)
    dY = np.random.default_rng(2).standard_normal((7, W.shape[1]))
    b1 = orc.backward(dY, W, A, B, scale, segs, f1["x_save"], f1["u_save"], n_rows=11, dropout=drop)
    b2 = orc.backward_blocked(dY, W, A, B, scale, segs, f1["x_save"], f1["u_save"], n_rows=11, dropout=drop)
    for key in ("dA", "dB", "dX", "V"):
        np.testing.assert_allclose(b2[key], b1[key], rtol=1e-12, atol=1e-12)


def test_ragged_ranks_equal_zero_padding():
    rng = np.random.default_rng(4)
    T, d_in, d_out = 9, 10, 6
    ranks = [1, 4, 2]
    A_list = [rng.standard_normal((r, d_in)) for r in ranks]
    B_list = [rng.standard_normal((r, d_out)) for r in ranks]
    X, W = rng.standard_normal((T, d_in)), rng.standard_normal((d_in, d_out))
    scale = np.array([8.0 / r for r in ranks])                      # alpha / r_a per adapter
    segs = np.array([(0, 3, 0, 1), (3, 3, 1, 0), (6, 3, 2, 1)])
    ragged = orc.forward_ragged(X, W, A_list, B_list, scale, segs)
    A_all, B_all = orc.pad_adapters(A_list, B_list, 4)
    padded = orc.forward(X, W, A_all, B_all, scale, segs)
    np.testing.assert_allclose(padded["Y"], ragged, rtol=1e-13, atol=1e-13)
    # brute force for one row of the rank-1 adapter
    t = 1
    y = X[t] @ W + scale[0] * float(A_list[0][0] @ X[t]) * B_list[0][0]
    np.testing.assert_allclose(ragged[t], y, rtol=1e-13)
    # gradients of the padding rows are exactly zero, those of the real rows match the ragged definition
    dY = rng.standard_normal((6, d_out))
    bwd = orc.backward(dY, W, A_all, B_all, scale, segs, padded["x_save"], padded["u_save"], n_rows=T)
    assert bwd["ft_adapters"] == [0, 2]
    assert not bwd["dA"][0, 1:].any() and not bwd["dB"][0, 1:].any()
    assert not bwd["dA"][1, 2:].any() and not bwd["dB"][1, 2:].any()
    g_rows = slice(0, 3)
    u = X[0:3] @ A_list[0].T
    np.testing.assert_allclose(bwd["dB"][0, :1], scale[0] * (u.T @ dY[g_rows]), rtol=1e-12)


def test_backward_ragged_is_the_gradient_of_forward_ragged():
    """L = sum(Y * dY_full) over the fine-tuning rows: every entry of dA, dB (own ranks, nothing padded) and dX
    against central finite differences of ``forward_ragged``; and the padded layer's gradients agree on the
    rows that exist."""
    rng = np.random.default_rng(14)
    T, d_in, d_out = 10, 7, 5
    ranks = [2, 5, 1, 3]
    A_list = [rng.standard_normal((r, d_in)) for r in ranks]
    B_list = [rng.standard_normal((r, d_out)) for r in ranks]
    X, W = rng.standard_normal((T, d_in)), rng.standard_normal((d_in, d_out))
    scale = np.array([4.0 / r for r in ranks])
    segs = np.array([(0, 2, 3, 1), (2, 3, 1, 0), (5, 2, 0, 1), (7, 3, 3, 1)])      # adapter 3 trains on two segments
    ft_rows = [0, 1, 5, 6, 7, 8, 9]                                               # save order = table order
    dY = rng.standard_normal((len(ft_rows), d_out))
    x_save = X[ft_rows]
    got = orc.backward_ragged(dY, W, A_list, B_list, scale, segs, x_save, n_rows=T)
    assert got["ft_adapters"] == [3, 0]

    def loss(Xv, Al, Bl):
        Y = orc.forward_ragged(Xv, W, Al, Bl, scale, segs)
        return float((Y[ft_rows] * dY).sum())

    eps = 1e-6
    for g, a in enumerate(got["ft_adapters"]):
        for name, lst, grad in (("A", A_list, got["dA"][g]), ("B", B_list, got["dB"][g])):
            num = np.zeros_like(grad)
            for idx in np.ndindex(*grad.shape):
                hi = [m.copy() for m in lst]; lo = [m.copy() for m in lst]
                hi[a][idx] += eps; lo[a][idx] -= eps
                args_hi = (hi, B_list) if name == "A" else (A_list, hi)
                args_lo = (lo, B_list) if name == "A" else (A_list, lo)
                num[idx] = (loss(X, *args_hi) - loss(X, *args_lo)) / (2 * eps)
            np.testing.assert_allclose(grad, num, rtol=1e-6, atol=1e-7)
    num = np.zeros((len(ft_rows), d_in))
    for m, t in enumerate(ft_rows):
        for k in range(d_in):
            hi, lo = X.copy(), X.copy()
            hi[t, k] += eps; lo[t, k] -= eps
            num[m, k] = (loss(hi, A_list, B_list) - loss(lo, A_list, B_list)) / (2 * eps)
    np.testing.assert_allclose(got["dX"], num, rtol=1e-6, atol=1e-7)
    # the zero-padded layer gives the same numbers where the rows exist
    A_all, B_all = orc.pad_adapters(A_list, B_list, 5)
    fwd = orc.forward(X, W, A_all, B_all, scale, segs)
    pad = orc.backward(dY, W, A_all, B_all, scale, segs, fwd["x_save"], fwd["u_save"], n_rows=T)
    assert pad["ft_adapters"] == got["ft_adapters"]
    for g, a in enumerate(got["ft_adapters"]):
        np.testing.assert_allclose(pad["dA"][g, :ranks[a]], got["dA"][g], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(pad["dB"][g, :ranks[a]], got["dB"][g], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(pad["dX"], got["dX"], rtol=1e-12, atol=1e-12)
