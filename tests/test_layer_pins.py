"""Pins for the decoder-layer oracle: hand values and defining properties of its pieces, causality,
sequence independence, the base-layer limit and finite differences."""
import math

import numpy as np
import pytest
import torch

from oracle import layer_oracle as lo

torch.manual_seed(0)
F64 = torch.float64


def make_params(d=16, ffn=24, r=2, n_ad=3, n_heads=4, n_kv=2, seed=0):
    g = torch.Generator().manual_seed(seed)
    dh = d // n_heads
    dims = {"q": (d, d), "k": (d, n_kv * dh), "v": (d, n_kv * dh), "o": (d, d), "gate": (d, ffn), "up": (d, ffn), "down": (ffn, d)}
    p = {"g1": 1.0 + 0.1 * torch.randn(d, generator=g, dtype=F64), "g2": 1.0 + 0.1 * torch.randn(d, generator=g, dtype=F64)}
    for name, (di, do) in dims.items():
        p["W_" + name] = torch.randn(di, do, generator=g, dtype=F64) / math.sqrt(di)
        p["A_" + name] = 0.3 * torch.randn(n_ad, r, di, generator=g, dtype=F64)
        p["B_" + name] = 0.3 * torch.randn(n_ad, r, do, generator=g, dtype=F64)
        p["s_" + name] = torch.tensor([2.0, 0.5, 1.0], dtype=F64)
    return p


def test_rmsnorm_hand_value_and_unit_rms():
    x = torch.tensor([[3.0, 4.0, 0.0, 0.0]], dtype=F64)            # mean square 25 / 4
    y = lo.rmsnorm(x, torch.ones(4, dtype=F64), eps=0.0)
    assert torch.allclose(y, torch.tensor([[1.2, 1.6, 0.0, 0.0]], dtype=F64))
    z = lo.rmsnorm(torch.randn(5, 32, dtype=F64), torch.ones(32, dtype=F64), eps=0.0)
    assert torch.allclose((z * z).mean(-1), torch.ones(5, dtype=F64))
    assert torch.allclose(lo.rmsnorm(x, 2 * torch.ones(4, dtype=F64), eps=0.0), 2 * y)


def test_rope_hand_value_norm_and_relative_position():
    # d_head 2, position 1: rotation by the angle 1 (theta^0)
    x = torch.tensor([[[1.0, 0.0]]], dtype=F64)
    y = lo.rope(x, torch.tensor([1]))
    assert torch.allclose(y, torch.tensor([[[math.cos(1.0), math.sin(1.0)]]], dtype=F64))
    q, k = torch.randn(1, 1, 8, dtype=F64), torch.randn(1, 1, 8, dtype=F64)
    assert torch.allclose(lo.rope(q, torch.tensor([7])).norm(), q.norm())
    dot = lambda m, n: float((lo.rope(q, torch.tensor([m])) * lo.rope(k, torch.tensor([n]))).sum())
    assert dot(5, 2) == pytest.approx(dot(13, 10), rel=1e-12) and dot(5, 2) != pytest.approx(dot(5, 3), rel=1e-6)
    assert torch.equal(lo.rope(q, torch.tensor([0])), q)


def test_attention_single_token_and_uniform_values():
    q, k, v = (torch.randn(3, 4, 4, dtype=F64) for _ in range(3))
    k, v = k[:, :2], v[:, :2]
    one = lo.attention(q, k, v, [[0], [1], [2]])                    # one-token sequences return their own value
    assert torch.allclose(one, v.repeat_interleave(2, dim=1))
    vv = torch.ones(3, 2, 4, dtype=F64) * 0.7                       # equal values: any softmax weights give them back
    assert torch.allclose(lo.attention(q, k, vv, [[0, 1, 2]]), torch.full((3, 4, 4), 0.7, dtype=F64))


def test_causality_and_sequence_independence():
    p = make_params()
    x = torch.randn(9, 16, dtype=F64)
    ra = [0, 0, 0, 1, 1, -1, 2, 2, 2]
    seqs = [[0, 1, 2], [3, 4], [5], [6, 7, 8]]
    y = lo.layer_forward(x, p, ra, seqs, 4, 2)
    x2 = x.clone(); x2[2] += 1.0                                     # a later token of sequence 0
    y2 = lo.layer_forward(x2, p, ra, seqs, 4, 2)
    assert torch.equal(y2[:2], y[:2]) and not torch.allclose(y2[2], y[2])
    assert torch.equal(y2[3:], y[3:])                                # other sequences never see it
    # the row order inside the batch does not matter, only membership and order inside a sequence
    perm = [6, 7, 8, 5, 3, 4, 0, 1, 2]
    yp = lo.layer_forward(x[perm], p, [ra[i] for i in perm], [[6, 7, 8], [4, 5], [3], [0, 1, 2]], 4, 2)
    assert torch.allclose(yp, y[perm], atol=1e-13)


def test_zero_b_is_the_base_layer():
    p = make_params()
    for name in lo.PROJ:
        p["B_" + name] = torch.zeros_like(p["B_" + name])
    x = torch.randn(6, 16, dtype=F64)
    y = lo.layer_forward(x, p, [0, 1, 2, 0, 1, 2], [[0, 1, 2], [3, 4, 5]], 4, 2)
    y0 = lo.layer_forward(x, p, [-1] * 6, [[0, 1, 2], [3, 4, 5]], 4, 2)
    assert torch.equal(y, y0)


def test_gradients_by_finite_differences():
    p = make_params(seed=3)
    x = torch.randn(7, 16, dtype=F64)
    ra = [0, 0, 0, 0, 2, 2, 2]
    seqs = [[0, 1, 2, 3], [4, 5, 6]]
    dy = torch.randn(7, 16, dtype=F64)
    g = lo.layer_backward(x, p, ra, seqs, 4, 2, dy, adapters=[0, 2])
    loss = lambda xx, pp: float((lo.layer_forward(xx, pp, ra, seqs, 4, 2) * dy).sum())
    h = 1e-6
    for name in ("q", "v", "gate", "down"):
        for slot, a in enumerate([0, 2]):
            for key, grad in (("A_", g["dA_" + name]), ("B_", g["dB_" + name])):
                idx = (a, 1, 3)
                pp, pm = dict(p), dict(p)
                pp[key + name] = p[key + name].clone(); pp[key + name][idx] += h
                pm[key + name] = p[key + name].clone(); pm[key + name][idx] -= h
                fd = (loss(x, pp) - loss(x, pm)) / (2 * h)
                assert float(grad[slot, 1, 3]) == pytest.approx(fd, rel=1e-5, abs=1e-8)
    for t, c in ((0, 0), (3, 5), (6, 15)):
        xp, xm = x.clone(), x.clone(); xp[t, c] += h; xm[t, c] -= h
        assert float(g["dx"][t, c]) == pytest.approx((loss(xp, p) - loss(xm, p)) / (2 * h), rel=1e-5, abs=1e-8)


# ---- wiring pins: each is written out as literals, so that a swapped operand, a dropped residual, a
# ---- missing softmax scale or a wrong head mapping in the oracle changes the expected numbers -----------
def _tiny_params(d, ffn, n_kv_cols):
    """One adapter slot with B = 0 (base layer only); every weight zero until a test fills it in."""
    z = lambda r, c: torch.zeros(r, c, dtype=F64)
    dims = {"q": (d, d), "k": (d, n_kv_cols), "v": (d, n_kv_cols), "o": (d, d), "gate": (d, ffn), "up": (d, ffn),
            "down": (ffn, d)}
    p = {"g1": torch.ones(d, dtype=F64), "g2": torch.ones(d, dtype=F64)}
    for name, (di, do) in dims.items():
        p["W_" + name] = z(di, do)
        p["A_" + name] = torch.zeros(1, 1, di, dtype=F64)
        p["B_" + name] = torch.zeros(1, 1, do, dtype=F64)
        p["s_" + name] = torch.ones(1, dtype=F64)
    return p


def test_all_projections_zero_returns_the_input():
    """Both residual connections: with every projection zero the layer is the identity."""
    p = _tiny_params(4, 6, 2)
    x = torch.randn(5, 4, dtype=F64)
    assert torch.equal(lo.layer_forward(x, p, [-1] * 5, [[0, 1, 2], [3, 4]], 2, 1), x)


def test_silu_gate_hand_value_tells_gate_from_up():
    """x = [1, -1] has unit RMS, so h2 = x (up to eps); gate gives g = [1, 2], up gives u = [3, -1], the down
    projection is the identity and the attention branch is zero:  y = x + [silu(1) 3, silu(2) (-1)].
    silu(1) = 0.7310585786300049, silu(2) = 1.7615941559557646.  (With gate and up swapped the second
    term would be [silu(3) 1, silu(-1) 2] = [2.8577, -0.5379].)"""
    p = _tiny_params(2, 2, 2)
    p["W_gate"] = torch.tensor([[1.0, 2.0], [0.0, 0.0]], dtype=F64)
    p["W_up"] = torch.tensor([[3.0, -1.0], [0.0, 0.0]], dtype=F64)
    p["W_down"] = torch.eye(2, dtype=F64)
    y = lo.layer_forward(torch.tensor([[1.0, -1.0]], dtype=F64), p, [-1], [[0]], 1, 1)
    want = torch.tensor([[1.0 + 3 * 0.7310585786300049, -1.0 - 1.7615941559557646]], dtype=F64)
    assert torch.allclose(y, want, atol=1e-4, rtol=0)


def test_attention_residual_hand_value():
    """One-token sequence, W_v = W_o = identity, no feed-forward:  y = x + RMSNorm(x) = 2 x for unit-RMS x."""
    p = _tiny_params(2, 2, 2)
    p["W_v"] = torch.eye(2, dtype=F64)
    p["W_o"] = torch.eye(2, dtype=F64)
    y = lo.layer_forward(torch.tensor([[1.0, -1.0]], dtype=F64), p, [-1], [[0]], 1, 1)
    assert torch.allclose(y, torch.tensor([[2.0, -2.0]], dtype=F64), atol=1e-4, rtol=0)


def test_attention_softmax_scale_hand_value():
    """Two tokens, one head of size 4: q1 . k1 = 2 ln 3 and q1 . k0 = 0, so with the 1 / sqrt(4) scale the scores
    of token 1 are (0, ln 3) and its weights (1/4, 3/4); without the scale they would be (1/10, 9/10)."""
    q = torch.tensor([[[0.0, 0, 0, 0]], [[2.0, 0, 0, 0]]], dtype=F64)
    k = torch.tensor([[[0.0, 0, 0, 0]], [[math.log(3.0), 0, 0, 0]]], dtype=F64)
    v = torch.tensor([[[1.0, 0, 0, 0]], [[0.0, 1, 0, 0]]], dtype=F64)
    out = lo.attention(q, k, v, [[0, 1]])
    assert torch.allclose(out[0, 0], torch.tensor([1.0, 0, 0, 0], dtype=F64))            # token 0 sees only itself
    assert torch.allclose(out[1, 0], torch.tensor([0.25, 0.75, 0, 0], dtype=F64), atol=1e-12)


def test_grouped_query_heads_read_their_own_kv_head():
    """Four query heads over two key-value heads: heads 0, 1 read kv head 0 and heads 2, 3 read kv head 1."""
    q = torch.randn(1, 4, 2, dtype=F64)
    k = torch.randn(1, 2, 2, dtype=F64)
    v = torch.tensor([[[1.0, 1.0], [2.0, 2.0]]], dtype=F64)          # kv head 0 is all ones, kv head 1 all twos
    out = lo.attention(q, k, v, [[0]])
    want = torch.tensor([[[1.0, 1.0], [1.0, 1.0], [2.0, 2.0], [2.0, 2.0]]], dtype=F64)
    assert torch.equal(out, want)
    # and the scores use the same mapping: two tokens, the key of kv head 1 at token 1 is large along the
    # query of head 2 only, so only heads 2 and 3 can prefer token 1 ... head 3's query is orthogonal to it
    q2 = torch.zeros(2, 4, 2, dtype=F64); q2[1, 2, 0] = 50.0
    k2 = torch.zeros(2, 2, 2, dtype=F64); k2[1, 1, 0] = 50.0
    v2 = torch.zeros(2, 2, 2, dtype=F64); v2[1, :, 1] = 1.0          # token 1 carries the marker in both kv heads
    out2 = lo.attention(q2, k2, v2, [[0, 1]])
    assert out2[1, 2, 1] > 0.999                                      # head 2 attends to token 1
    assert torch.allclose(out2[1, [0, 1, 3], 1], torch.full((3,), 0.5, dtype=F64))   # the others split evenly


def test_lora_linear_is_the_hot_path_oracle():
    """The layer oracle's projection equals the layer-free oracle of the hot path on a mixed table."""
    from oracle import mlora_oracle as orc
    rng = np.random.default_rng(5)
    T, d_in, d_out, r, n = 11, 6, 5, 2, 3
    X, W = rng.standard_normal((T, d_in)), rng.standard_normal((d_in, d_out))
    A, B = rng.standard_normal((n, r, d_in)), rng.standard_normal((n, r, d_out))
    s = np.array([2.0, 0.5, 1.25])
    segs = np.array([[0, 3, 1, 0], [3, 2, -1, 0], [5, 4, 0, 1], [10, 1, 2, 0]], dtype=np.int32)   # row 9 uncovered
    ref = orc.forward(X, W, A, B, s, segs)["Y"]
    ra = [1, 1, 1, -1, -1, 0, 0, 0, 0, -1, 2]
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    got = lo.lora_linear(t(X), t(W), t(A), t(B), t(s), ra)
    assert np.allclose(got.numpy(), ref, rtol=1e-12, atol=1e-12)
