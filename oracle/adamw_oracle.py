"""CPU oracle for the AdamW update of the fine-tuned adapters (TEST INFRASTRUCTURE ONLY).

Section 3.2 ("Backward subprocess") has the backward apply optimizer updates directly to the
shared adapter weights; Section 5 ("Fine-tuning Workload") fixes the optimizer: AdamW with
learning rate 1e-3 and weight decay 0.01.  The paper gives no betas or epsilon; the usual defaults
(0.9, 0.999, 1e-8) are taken.  This is the decoupled-weight-decay Adam step written out in fp64:

    theta <- theta - lr * wd * theta
    m     <- beta1 m + (1 - beta1) g
    v     <- beta2 v + (1 - beta2) g^2
    theta <- theta - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)         t = 1, 2, ...

Pins (tests/test_adamw_pins.py): torch.optim.AdamW in float64 over several steps (a library
routine), the closed form of the first step, pure decay under a zero gradient, and the bound
|delta theta| <= lr (1 + wd |theta|) per step.  It shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def adamw_step(theta, g, m, v, step: int, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999,
               eps: float = 1e-8, weight_decay: float = 0.01):
    """One update; `step` is the 1-based index of this update.  Returns new (theta, m, v) as float64."""
    theta = np.asarray(theta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    theta = theta - lr * weight_decay * theta
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    theta = theta - lr * m_hat / (np.sqrt(v_hat) + eps)
    return theta, m, v
