"""GPU parity of the layer with a real-valued zero-point (App. K: "zero-points only" and "both
zero-points and quantization scales"), against the oracle's *_zf functions."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import adamw_scale_tol, assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def _layer(seed, N, K, T, bits, g):
    d = synth.custom(seed, N, K, T, bits, g, outliers=True, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    rng = np.random.default_rng(seed)
    # trained zero-points: off the grid, some of them beyond the code range
    zf = (zeros.astype(np.float32) + rng.uniform(-1.3, 1.3, size=zeros.shape).astype(np.float32))
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    return d, packed, zeros, zf, scales, qw


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 0), (3, 64), (4, 128), (3, 32), (4, 256)])
def test_forward_and_backward_match_oracle(bits, g):
    N, K, T = 328, 768, 300
    d, packed, zeros, zf, scales, qw = _layer(500 + bits + g, N, K, T, bits, g)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    zf_d = torch.from_numpy(zf).cuda()
    Y = binding.qlinear_fwd_zf(qw, zf_d, X)
    dX, dS, dZ = binding.qlinear_bwd_zf(qw, zf_d, X, dY)
    binding.check_status()
    assert_close(dev_to_f64(Y), oracle.fwd_zf(d["X"], packed, zf, scales, bits, g), "Y")
    assert_close(dev_to_f64(dX), oracle.bwd_dx_zf(d["dY"], packed, zf, scales, K, bits, g), "dX")
    assert_close(dev_to_f64(dS), oracle.bwd_ds_zf(d["X"], d["dY"], packed, zf, bits, g), "dS")
    assert_close(dev_to_f64(dZ), oracle.bwd_dz(d["X"], d["dY"], scales, g), "dZ")


@pytest.mark.parametrize("bits,g", [(3, 0), (3, 64), (4, 192)])
def test_in_features_not_a_multiple_of_128(bits, g):
    # 3-bit rows without a 16-byte pitch take the single-CTA kernels
    N, K, T = 264, 576, 150
    d, packed, zeros, zf, scales, qw = _layer(600 + bits + g, N, K, T, bits, g)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    zf_d = torch.from_numpy(zf).cuda()
    Y = binding.qlinear_fwd_zf(qw, zf_d, X)
    dX, dS, dZ = binding.qlinear_bwd_zf(qw, zf_d, X, dY)
    binding.check_status()
    assert_close(dev_to_f64(Y), oracle.fwd_zf(d["X"], packed, zf, scales, bits, g), "Y")
    assert_close(dev_to_f64(dX), oracle.bwd_dx_zf(d["dY"], packed, zf, scales, K, bits, g), "dX")
    assert_close(dev_to_f64(dS), oracle.bwd_ds_zf(d["X"], d["dY"], packed, zf, bits, g), "dS")


def test_integral_zero_point_agrees_with_the_integer_path():
    d, packed, zeros, zf, scales, qw = _layer(7, 256, 512, 200, 3, 128)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    zi = torch.from_numpy(zeros.astype(np.float32)).cuda()
    Y0 = binding.qlinear_fwd(qw, X)
    Y1 = binding.qlinear_fwd_zf(qw, zi, X)
    dX0, dS0 = binding.qlinear_bwd(qw, X, dY)
    dX1, dS1, dZ1 = binding.qlinear_bwd_zf(qw, zi, X, dY)
    _, dZ0 = binding.qlinear_bwd_dsdz(qw, X, dY)
    binding.check_status()
    # delta = 0: the fused multiply-add adds an exact zero, so the operands are the same bits
    assert torch.equal(Y0, Y1) and torch.equal(dX0, dX1)
    assert torch.equal(dS0, dS1) and torch.equal(dZ0, dZ1)


@pytest.mark.parametrize("mode", ["scales only", "zero-points only", "both"])
@pytest.mark.parametrize("bits,g", [(4, 0), (3, 64)])
def test_one_training_step_of_each_mode(mode, bits, g):
    """App. K's three ablation modes: forward, backward, AdamW on what the mode trains."""
    N, K, T = 264, 512, 260
    d, packed, zeros, zf, scales, qw = _layer(900 + bits + g, N, K, T, bits, g)
    if mode == "scales only":
        zf = zeros.astype(np.float32)          # the zero-points stay the stored integers
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    zf_d = torch.from_numpy(zf.copy()).cuda()
    Y = binding.qlinear_fwd_zf(qw, zf_d, X)
    dX, dS, dZ = binding.qlinear_bwd_zf(qw, zf_d, X, dY)
    assert_close(dev_to_f64(Y), oracle.fwd_zf(d["X"], packed, zf, scales, bits, g), "Y")
    assert_close(dev_to_f64(dX), oracle.bwd_dx_zf(d["dY"], packed, zf, scales, K, bits, g), "dX")
    lr, b1, b2, eps = (float(np.float32(x)) for x in (1e-4, 0.9, 0.999, 1e-8))
    zero = np.zeros_like(scales)
    if mode in ("scales only", "both"):
        g_host = dS.cpu().numpy()
        m, v = torch.zeros_like(qw.scales), torch.zeros_like(qw.scales)
        binding.scale_adamw(qw.scales, dS, m, v, lr)
        so, _, _ = oracle.adamw(scales, g_host, zero, zero, lr, b1, b2, eps, 0.0, 1)
        got = qw.scales.cpu().numpy().astype(np.float64).ravel()
        assert np.all(np.abs(got - so) <= adamw_scale_tol(scales, g_host, zero, zero, lr, b1, b2, eps, 0.0, 1))
    if mode in ("zero-points only", "both"):
        g_host = dZ.cpu().numpy()
        m, v = torch.zeros_like(zf_d), torch.zeros_like(zf_d)
        binding.zero_adamw(zf_d, dZ, m, v, lr)
        zo, _, _ = oracle.adamw(zf, g_host, zero, zero, lr, b1, b2, eps, 0.0, 1)
        got = zf_d.cpu().numpy().astype(np.float64).ravel()
        assert np.all(np.abs(got - zo) <= adamw_scale_tol(zf, g_host, zero, zero, lr, b1, b2, eps, 0.0, 1))
        assert not np.array_equal(zf_d.cpu().numpy(), zf)
    binding.check_status()
    # the updated parameters feed the next forward
    s_new = qw.scales.cpu().numpy()
    z_new = zf_d.cpu().numpy()
    Y2 = binding.qlinear_fwd_zf(qw, zf_d, X)
    binding.check_status()
    assert_close(dev_to_f64(Y2), oracle.fwd_zf(d["X"], packed, z_new, s_new, bits, g), "Y after the step")
