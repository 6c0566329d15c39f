"""GPU parity: AdamW on the scales (App. A) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 1000, 131072 + 3])
@pytest.mark.parametrize("step,wd", [(1, 0.0), (7, 0.01), (1000, 0.0)])
def test_adamw_step(n, step, wd):
    rng = np.random.default_rng(n + step)
    s = (rng.random(n) * 0.01 + 1e-3).astype(np.float32)
    g = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    m = (rng.standard_normal(n) * 1e-3).astype(np.float32) if step > 1 else np.zeros(n, np.float32)
    v = (rng.random(n) * 1e-5).astype(np.float32) if step > 1 else np.zeros(n, np.float32)
    # the C ABI takes binary32 hyper-parameters: give the oracle exactly those values
    lr, b1, b2, eps, wd = (float(np.float32(x)) for x in (1e-5, 0.9, 0.999, 1e-8, wd))
    so, mo, vo = oracle.adamw(s, g, m, v, lr, b1, b2, eps, wd, step)
    ds, dg, dm, dv = (torch.from_numpy(a).cuda() for a in (s, g, m, v))
    binding.scale_adamw(ds, dg, dm, dv, lr, 0.9, 0.999, 1e-8, wd, step)
    torch.cuda.synchronize()
    got_s, got_m, got_v = (t.cpu().numpy().astype(np.float64) for t in (ds, dm, dv))
    # binary32 evaluation: the update term (<= ~lr/(1-b1) in size) carries a few ulps of
    # relative error, and the final s is rounded once to binary32
    assert np.all(np.abs(got_s - so) <= 1e-5 * lr * 10 + 2.0 ** -23 * np.abs(so))
    # m and v are two-term binary32 sums: a few ulps of the larger term (m may cancel)
    ulp = 2.0 ** -23
    gd, md, vd = (a.astype(np.float64) for a in (g, m, v))
    assert np.all(np.abs(got_m - mo) <= 3 * ulp * (np.abs(b1 * md) + np.abs((1 - b1) * gd)) + 1e-30)
    assert np.all(np.abs(got_v - vo) <= 4 * ulp * (np.abs(b2 * vd) + np.abs((1 - b2) * gd * gd)) + 1e-30)


def test_zero_gradient_and_first_step_sign():
    s = torch.full((64,), 0.5, device="cuda")
    z = torch.zeros(64, device="cuda")
    m, v = torch.zeros(64, device="cuda"), torch.zeros(64, device="cuda")
    binding.scale_adamw(s, z, m, v, 1e-3)
    assert torch.all(s == 0.5)
    g = torch.linspace(-1, 1, 64, device="cuda")
    g[g == 0] = 0.5
    binding.scale_adamw(s, g, m, v, 1e-3)
    torch.cuda.synchronize()
    assert torch.allclose(s, 0.5 - 1e-3 * torch.sign(g), atol=1e-7)
