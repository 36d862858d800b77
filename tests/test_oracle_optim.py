"""Pins for the optimizer oracle: torch's own clip + AdamW in fp64, and the first step's closed form."""
import numpy as np
import pytest
import torch

from oracle import optim_oracle as oo


@pytest.mark.parametrize("wd,max_norm", [(0.0, 2.0), (0.01, 0.05), (0.0, 0.0)])
def test_adamw_matches_torch(wd, max_norm):
    rng = np.random.default_rng(0)
    shapes = {"a": (7, 5), "b": (11,), "c": (3, 4, 2)}
    params = {k: rng.standard_normal(s) for k, s in shapes.items()}
    tp = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    opt = torch.optim.AdamW(list(tp.values()), lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    m = {k: np.zeros(s) for k, s in shapes.items()}
    v = {k: np.zeros(s) for k, s in shapes.items()}
    for step in range(1, 6):
        grads = {k: rng.standard_normal(s) * (0.01 if step % 2 else 3.0) for k, s in shapes.items()}
        for k in tp:
            tp[k].grad = torch.tensor(grads[k], dtype=torch.float64)
        if max_norm > 0:
            tn = float(torch.nn.utils.clip_grad_norm_(list(tp.values()), max_norm))
        norm = oo.adamw_step(params, grads, m, v, step, lr=1e-2, weight_decay=wd, max_norm=max_norm)
        opt.step()
        if max_norm > 0:
            assert norm == pytest.approx(tn, rel=1e-12)
        for k in params:
            assert np.allclose(params[k], tp[k].detach().numpy(), rtol=1e-12, atol=1e-14), (step, k)


def test_first_step_moves_every_weight_by_lr_against_the_gradient_sign():
    # step 1 without clipping or decay: m_hat = g, v_hat = g^2  =>  update = lr * g / (|g| + eps)
    g = {"w": np.array([0.5, -2.0, 1e-3])}
    p = {"w": np.zeros(3)}
    m = {"w": np.zeros(3)}
    v = {"w": np.zeros(3)}
    oo.adamw_step(p, g, m, v, 1, lr=1e-5, max_norm=0.0)
    assert np.allclose(p["w"], -1e-5 * np.sign(g["w"]), rtol=1e-4)
    assert oo.clip_coefficient(4.0, 2.0) == pytest.approx(0.5, rel=1e-6) and oo.clip_coefficient(1.0, 2.0) == 1.0
