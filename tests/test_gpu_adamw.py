"""GPU parity: AdamW on the scales (App. A) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding
from gpu_util import adamw_scale_tol

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
    assert np.all(np.abs(got_s - so) <= adamw_scale_tol(s, g, m, v, lr, b1, b2, eps, wd, step))
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


@pytest.mark.parametrize("bits,g", [(3, 128), (4, 64), (3, 32), (4, 0), (3, 256)])
def test_step_applied_where_ds_is_produced_equals_the_two_calls(bits, g):
    """peqa_qlinear_bwd_ds_adamw against peqa_qlinear_bwd followed by peqa_scale_adamw:
    the same bits in dS, scales, m and v, for groups that the dS kernel finishes itself
    (g <= 128) and for those that go through the reduction kernel."""
    from paper_2305_14152_b200 import synth
    from gpu_util import bf16_to_dev, oracle_layer, to_qweight
    N, K, T = 328, 768, 300
    d = synth.custom(800 + bits + g, N, K, T, bits, g, outliers=True, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    G = scales.shape[1]
    rng = np.random.default_rng(3)
    m0 = (rng.standard_normal((N, G)) * 1e-3).astype(np.float32)
    v0 = (rng.random((N, G)) * 1e-5).astype(np.float32)
    out = []
    for fused in (False, True):
        qw = to_qweight(packed, zeros, scales.copy(), bits, g, K)
        m, v = torch.from_numpy(m0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
        if fused:
            dS = binding.qlinear_bwd_ds_adamw(qw, X, dY, m, v, 1e-4, weight_decay=0.01, step=7)
        else:
            dS = binding.qlinear_bwd(qw, X, dY, need_dx=False)[1]
            binding.scale_adamw(qw.scales, dS, m, v, 1e-4, 0.9, 0.999, 1e-8, 0.01, 7)
        torch.cuda.synchronize()
        out.append((dS.clone(), qw.scales.clone(), m, v))
    binding.check_status()
    for a, b in zip(out[0], out[1]):
        assert torch.equal(a, b)
    assert not torch.equal(out[0][1].cpu(), torch.from_numpy(scales))      # the scales did move
