"""Pins of the checker's AdamW step and learning-rate rebound (the optimizer of the paper's experiments;
Methodology, "learning rate rebound") against torch.optim.AdamW and closed forms.  CPU only."""
import numpy as np
import torch

from oracle import ab_oracle as orc


def test_adamw_matches_the_library_optimizer():
    rng = np.random.default_rng(0)
    p0 = rng.standard_normal(257)
    grads = [rng.standard_normal(257) for _ in range(6)]
    lrs = [1e-3, 2e-3, 5e-4, 1e-3, 1e-3, 3e-3]
    t = torch.nn.Parameter(torch.tensor(p0, dtype=torch.float64))
    opt = torch.optim.AdamW([t], lr=1e-3, betas=(0.9, 0.98), eps=1e-6, weight_decay=0.05)
    p, m, v = p0.copy(), np.zeros(257), np.zeros(257)
    for k, (g, lr) in enumerate(zip(grads, lrs), start=1):
        for grp in opt.param_groups:
            grp["lr"] = lr
        t.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        p, m, v = orc.adamw_step(p, g, m, v, lr, k, 0.9, 0.98, 1e-6, 0.05)
        assert np.allclose(p, t.detach().numpy(), rtol=1e-12, atol=1e-14), k


def test_adamw_first_step_closed_form():
    # m = (1-b1) g and v = (1-b2) g^2 make the bias-corrected ratio g / |g|: a step of exactly lr against the
    # sign of the gradient (for eps -> 0), after the decay
    p = np.array([1.0, -2.0, 0.5])
    g = np.array([0.3, -4.0, 1e-3])
    out, m, v = orc.adamw_step(p, g, np.zeros(3), np.zeros(3), 0.1, 1, eps=1e-30, weight_decay=0.5)
    assert np.allclose(out, p * (1 - 0.05) - 0.1 * np.sign(g), rtol=1e-12)
    assert np.allclose(m, 0.1 * g) and np.allclose(v, 0.001 * g * g)
    # zero gradient, zero state: only the decay acts
    out, _, _ = orc.adamw_step(p, np.zeros(3), np.zeros(3), np.zeros(3), 0.1, 1, weight_decay=0.5)
    assert np.allclose(out, 0.95 * p)


def test_lr_rebound_factor():
    assert orc.lr_rebound_factor(0, 10, 0.0) == 0.0
    assert orc.lr_rebound_factor(5, 10, 0.0) == 0.5
    assert orc.lr_rebound_factor(10, 10, 0.0) == 1.0 and orc.lr_rebound_factor(99, 10, 0.2) == 1.0
    assert abs(orc.lr_rebound_factor(5, 10, 0.2) - 0.6) < 1e-15
    assert orc.lr_rebound_factor(3, 0, 0.1) == 1.0          # no rebound configured
    f = [orc.lr_rebound_factor(k, 7, 0.01) for k in range(9)]
    assert all(b >= a for a, b in zip(f, f[1:])) and f[0] == 0.01 and f[-1] == 1.0
