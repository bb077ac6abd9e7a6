"""Pins for the AdamW oracle: a library optimizer in float64, the closed form of the first step,
pure decay under zero gradients, and the per-step bound on the update."""
import numpy as np
import torch

from oracle import adamw_oracle as ao


def test_matches_torch_adamw_float64_over_steps():
    rng = np.random.default_rng(0)
    theta0 = rng.standard_normal((3, 7))
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    theta, m, v = theta0.copy(), np.zeros_like(theta0), np.zeros_like(theta0)
    for step in range(1, 6):
        g = rng.standard_normal(theta0.shape) * 10.0 ** rng.integers(-3, 2)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        theta, m, v = ao.adamw_step(theta, g, m, v, step)
        np.testing.assert_allclose(theta, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_first_step_closed_form():
    theta = np.array([2.0, -1.0, 0.5])
    g = np.array([0.3, -4.0, 1e-3])
    lr, wd, eps = 1e-3, 0.01, 1e-8
    new, m, v = ao.adamw_step(theta, g, np.zeros(3), np.zeros(3), 1, lr=lr, eps=eps, weight_decay=wd)
    # after bias correction m_hat = g and v_hat = g^2 exactly
    expect = theta * (1 - lr * wd) - lr * g / (np.abs(g) + eps)
    np.testing.assert_allclose(new, expect, rtol=1e-13)
    np.testing.assert_allclose(m, 0.1 * g, rtol=1e-13)
    np.testing.assert_allclose(v, 0.001 * g * g, rtol=1e-13)


def test_zero_gradient_is_pure_decay():
    theta = np.array([1.0, -3.0])
    m = v = np.zeros(2)
    for step in range(1, 4):
        theta, m, v = ao.adamw_step(theta, np.zeros(2), m, v, step)
    np.testing.assert_allclose(theta, np.array([1.0, -3.0]) * (1 - 1e-5) ** 3, rtol=1e-13)
    assert not m.any() and not v.any()


def test_update_is_bounded_by_lr():
    rng = np.random.default_rng(1)
    theta = rng.standard_normal(1000)
    m, v = np.zeros(1000), np.zeros(1000)
    for step in range(1, 5):
        g = rng.standard_normal(1000) * 100
        new, m, v = ao.adamw_step(theta, g, m, v, step)
        # |m_hat| / sqrt(v_hat) <= 1 / sqrt(1 - beta2) in general and about 1 for fresh moments
        assert np.all(np.abs(new - theta) <= 1e-3 * (0.01 * np.abs(theta) + 1.0 / np.sqrt(1 - 0.999)) + 1e-12)
        theta = new
