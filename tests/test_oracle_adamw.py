"""Pins for the oracle's AdamW step on the scales (optimizer named in the paper's App. A)."""
import numpy as np
import torch

import oracle


def test_first_step_closed_form():
    rng = np.random.default_rng(0)
    s = rng.random(64, dtype=np.float32) + 0.5
    g = rng.standard_normal(64).astype(np.float32)
    z = np.zeros(64, np.float32)
    lr, eps = 1e-3, 1e-8
    so, mo, vo = oracle.adamw(s, g, z, z, lr, 0.9, 0.999, eps, 0.0, 1)
    gd = g.astype(np.float64)
    np.testing.assert_allclose(so, s.astype(np.float64) - lr * gd / (np.abs(gd) + eps), rtol=1e-13)
    np.testing.assert_allclose(mo, 0.1 * gd, rtol=1e-12)
    np.testing.assert_allclose(vo, 0.001 * gd * gd, rtol=1e-9)


def test_zero_gradient_leaves_scale_unchanged_without_decay():
    s = np.array([0.25, 1.5], np.float32)
    z = np.zeros(2, np.float32)
    so, mo, vo = oracle.adamw(s, z, z, z, 1e-2, step=3)
    assert np.array_equal(so, s.astype(np.float64)) and not mo.any() and not vo.any()
    so, _, _ = oracle.adamw(s, z, z, z, 1e-2, weight_decay=0.1, step=3)
    np.testing.assert_allclose(so, s.astype(np.float64) * (1 - 1e-3), rtol=1e-15)


def test_ten_steps_against_torch_adamw_float64():
    rng = np.random.default_rng(1)
    n = 33
    s0 = (rng.random(n) + 0.5).astype(np.float32)
    grads = [rng.standard_normal(n).astype(np.float32) for _ in range(10)]
    p = torch.tensor(s0.astype(np.float64), requires_grad=True)
    opt = torch.optim.AdamW([p], lr=3e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    s = s0.astype(np.float64)
    m = np.zeros(n)
    v = np.zeros(n)
    for k, g in enumerate(grads, start=1):
        p.grad = torch.tensor(g.astype(np.float64))
        opt.step()
        # the oracle's state interface is fp32; keep the trajectory in fp64 by
        # feeding it values that are exactly representable only at step 1, and
        # compare one step at a time from torch's own state afterwards
        so, mo, vo = oracle.adamw(s.astype(np.float32), g, m.astype(np.float32), v.astype(np.float32),
                                  3e-4, 0.9, 0.999, 1e-8, 0.01, k)
        st = opt.state[p]
        np.testing.assert_allclose(so, p.detach().numpy(), rtol=2e-7)
        np.testing.assert_allclose(mo, st["exp_avg"].numpy(), rtol=2e-6, atol=1e-9)
        np.testing.assert_allclose(vo, st["exp_avg_sq"].numpy(), rtol=2e-6, atol=1e-12)
        s, m, v = p.detach().numpy().copy(), st["exp_avg"].numpy().copy(), st["exp_avg_sq"].numpy().copy()
