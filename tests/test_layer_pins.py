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
