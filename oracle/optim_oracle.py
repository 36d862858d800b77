"""CPU oracle for the optimizer step that follows the actor update (App. E: AdamW, constant learning rate
1e-5, betas (0.9, 0.999), weight decay 0, gradient clipping at 2.0), in fp64.

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path.

Parity status: pinned against torch.nn.utils.clip_grad_norm_ + torch.optim.AdamW in fp64
(tests/test_oracle_optim.py) and by the closed form of the first step.

Readings where the paper is silent: the clip is on the global L2 norm over all parameters with the
usual guard, coefficient = min(1, max_norm / (norm + 1e-6)); Adam epsilon = 1e-8; decoupled weight decay.
"""
from __future__ import annotations

import math
from typing import Dict

import numpy as np


def global_norm(grads: Dict[str, np.ndarray]) -> float:
    total = 0.0
    for k in grads:
        g = np.asarray(grads[k], dtype=np.float64)
        total += float(np.sum(g * g))
    return math.sqrt(total)


def clip_coefficient(norm: float, max_norm: float) -> float:
    return min(1.0, max_norm / (norm + 1e-6))


def adamw_step(params, grads, m, v, step: int, lr=1e-5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0,
               max_norm=2.0):
    """One update, in place on the fp64 dicts params / m / v; `step` counts from 1.  Returns the gradient
    norm before clipping."""
    norm = global_norm(grads)
    coef = clip_coefficient(norm, max_norm) if max_norm > 0 else 1.0
    bc1 = 1.0 - beta1 ** step
    bc2 = 1.0 - beta2 ** step
    for k in params:
        g = np.asarray(grads[k], dtype=np.float64) * coef
        m[k] = beta1 * m[k] + (1.0 - beta1) * g
        v[k] = beta2 * v[k] + (1.0 - beta2) * g * g
        m_hat = m[k] / bc1
        v_hat = v[k] / bc2
        params[k] = params[k] - lr * (m_hat / (np.sqrt(v_hat) + eps) + weight_decay * params[k])
    return norm
