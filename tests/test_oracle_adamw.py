"""Pins of the oracle's AdamW step on the factors: the trajectory of torch.optim.AdamW in float64 (a library
routine with the published algorithm), and two closed forms."""
import numpy as np
import torch

import oracle


def test_matches_torch_adamw_over_several_steps():
    rng = np.random.default_rng(0)
    n, steps = 224, 6
    s0 = rng.uniform(0.01, 0.2, n)
    grads = [rng.normal(0, 50, n) for _ in range(steps)]
    p = torch.nn.Parameter(torch.tensor(s0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=2e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    s, m, v = s0.copy(), np.zeros(n), np.zeros(n)
    for t, g in enumerate(grads, start=1):
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        s, m, v = oracle.adamw_step(s, g, m, v, t)
        assert np.allclose(s, p.detach().numpy(), rtol=1e-12, atol=1e-15)


def test_first_step_moves_by_lr_against_the_sign_of_the_gradient():
    # step 1: m_hat = g, v_hat = g^2, so the update is lr * (g / (|g| + eps) + wd * s)
    s = np.array([0.5, 0.5, -0.25])
    g = np.array([3.0, -7.0, 1e-3])
    s1, m, v = oracle.adamw_step(s, g, np.zeros(3), np.zeros(3), 1, lr=1e-2, weight_decay=0.0)
    assert np.allclose(s1, s - 1e-2 * np.sign(g), atol=1e-6)
    assert np.allclose(m, 0.1 * g) and np.allclose(v, 0.001 * g * g)


def test_zero_gradient_leaves_only_the_weight_decay():
    s = np.array([0.2, -0.4])
    s1, m, v = oracle.adamw_step(s, np.zeros(2), np.zeros(2), np.zeros(2), 1, lr=1e-3, weight_decay=0.1)
    assert np.allclose(s1, s * (1 - 1e-4)) and not m.any() and not v.any()
