"""Pins for the oracle's optimiser on the coefficients (Adam with decoupled decay, cosine
schedule) and for the fixed-weight averages: closed forms and PyTorch's own CPU optimiser."""

import numpy as np
import torch

from oracle import twa_oracle as orc


def test_adam_first_step_is_a_signed_step_of_size_lr():
    c = np.array([3.0, -0.25, 1e-3, -7.0])
    a, m, v = orc.adam_update(np.zeros(4), np.zeros(4), np.zeros(4), c, lr=0.01, t=1, eps=0.0)
    np.testing.assert_allclose(a, -0.01 * np.sign(c), rtol=1e-15)
    np.testing.assert_allclose(m, 0.1 * c, rtol=1e-15)
    np.testing.assert_allclose(v, 0.001 * c * c, rtol=1e-12)


def test_adam_constant_gradient_keeps_unit_steps_and_decay_is_decoupled():
    c = np.array([2.0, -5.0])
    a, m, v = np.array([1.0, 1.0]), np.zeros(2), np.zeros(2)
    for t in range(1, 6):
        a_prev = a
        a, m, v = orc.adam_update(a, m, v, c, lr=0.1, t=t, eps=0.0, weight_decay=0.5)
        # bias-corrected moments of a constant gradient are the gradient itself: step = lr * sign
        np.testing.assert_allclose(a, a_prev * (1 - 0.1 * 0.5) - 0.1 * np.sign(c), rtol=1e-13)


def test_adam_matches_torch_adamw_over_steps():
    rng = np.random.default_rng(0)
    n, steps = 17, 12
    alpha0 = rng.standard_normal(n)
    grads = rng.standard_normal((steps, n)) * np.logspace(-3, 1, n)
    p = torch.nn.Parameter(torch.tensor(alpha0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=0.01, betas=(0.9, 0.98), eps=1e-9, weight_decay=0.01)
    a, m, v = alpha0.copy(), np.zeros(n), np.zeros(n)
    for t in range(steps):
        p.grad = torch.tensor(grads[t], dtype=torch.float64)
        opt.step()
        a, m, v = orc.adam_update(a, m, v, grads[t], lr=0.01, t=t + 1, beta1=0.9, beta2=0.98, eps=1e-9,
                                  weight_decay=0.01)
        np.testing.assert_allclose(a, p.detach().numpy(), rtol=1e-12, atol=1e-14)
    # plain Adam (no decay) against torch.optim.Adam
    q = torch.nn.Parameter(torch.tensor(alpha0, dtype=torch.float64))
    opt2 = torch.optim.Adam([q], lr=0.003)
    a, m, v = alpha0.copy(), np.zeros(n), np.zeros(n)
    for t in range(steps):
        q.grad = torch.tensor(grads[t], dtype=torch.float64)
        opt2.step()
        a, m, v = orc.adam_update(a, m, v, grads[t], lr=0.003, t=t + 1)
    np.testing.assert_allclose(a, q.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_cosine_schedule_end_points_midpoint_and_library():
    assert orc.cosine_lr(0.01, 0, 100) == 0.01
    assert abs(orc.cosine_lr(0.01, 100, 100)) < 1e-18
    np.testing.assert_allclose(orc.cosine_lr(0.01, 50, 100), 0.005, rtol=1e-14)
    np.testing.assert_allclose(orc.cosine_lr(0.01, 25, 100, min_lr=0.002), 0.002 + 0.008 * (1 + np.sqrt(0.5)) / 2,
                               rtol=1e-14)
    p = torch.nn.Parameter(torch.zeros(1))
    opt = torch.optim.SGD([p], lr=0.01)
    sched = torch.optim.lr_scheduler.CosineAnnealingLR(opt, T_max=40, eta_min=1e-4)
    for step in range(41):
        np.testing.assert_allclose(orc.cosine_lr(0.01, step, 40, 1e-4), sched.get_last_lr()[0], rtol=1e-9)
        opt.step()
        sched.step()


def test_weighted_average_special_cases():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((300, 6)).astype(np.float32)
    # equal weights: the mean (SWA); weights on the last t: LAWA
    np.testing.assert_allclose(orc.weighted_average(W, np.full(6, 1 / 6)), orc.mean(W), rtol=1e-14, atol=1e-16)
    lawa = np.array([0, 0, 0, 1 / 3, 1 / 3, 1 / 3])
    np.testing.assert_allclose(orc.weighted_average(W, lawa), W[:, 3:].astype(np.float64).mean(axis=1), rtol=1e-13,
                               atol=1e-16)
    # geometric weights: the recursion e <- d e + (1-d) w_i started at w_0
    d = 0.7
    e = W[:, 0].astype(np.float64)
    for i in range(1, 6):
        e = d * e + (1 - d) * W[:, i].astype(np.float64)
    wts = np.array([d ** 5] + [(1 - d) * d ** (5 - i) for i in range(1, 6)])
    np.testing.assert_allclose(orc.weighted_average(W, wts), e, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(orc.weighted_average(W, wts), W.astype(np.float64) @ wts, rtol=1e-13, atol=1e-15)
