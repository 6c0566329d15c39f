"""GPU parity: RTN quantization (Eq. 1) and the packed layout, bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import u32

pytestmark = pytest.mark.gpu


def _compare(W, bits, g):
    codes, zeros, scales = oracle.quantize_rtn(W, bits, g)
    packed = oracle.pack(codes, bits)
    qw = binding.quantize_rtn(torch.from_numpy(W).cuda(), bits, g)
    torch.cuda.synchronize()
    assert np.array_equal(qw.scales.cpu().numpy().view(np.uint32), scales.view(np.uint32))
    assert np.array_equal(qw.zeros.cpu().numpy(), zeros)
    assert np.array_equal(u32(qw.qweight), packed)
    un = binding.unpack(qw.qweight, W.shape[1], bits)
    assert np.array_equal(un.cpu().numpy(), codes)


def test_c1_toy_layer():
    d = next(synth.generate("c1"))
    _compare(d["W"], 4, 0)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("g", [0, 32, 64, 128, 256])
def test_group_sizes_and_ragged_rows(bits, g):
    d = synth.custom(17 + bits + g, 203, 768, 1, bits, g, outliers=True)
    _compare(d["W"], bits, g)


def test_c2_shape_three_bit_g128_with_outliers():
    d = next(synth.generate("c2", T=1))
    _compare(d["W"], 3, 128)


def test_wide_rows_per_channel():
    d = synth.custom(5, 64, 22016, 1, 3, 0, sigma_w=0.015)
    _compare(d["W"], 3, 0)
    d = synth.custom(6, 48, 11008, 1, 4, 0)
    _compare(d["W"], 4, 0)


def test_degenerate_rows():
    W = np.zeros((8, 64), np.float32)
    W[0, :] = 0.25
    W[1, :] = np.linspace(1.0, 2.0, 64)
    W[2, :] = -np.linspace(1.0, 2.0, 64)
    W[3, 1:] = np.arange(1, 64, dtype=np.float32)
    W[3, 0] = -0.0
    W[4, :] = np.float32(1e-30) * np.arange(64)
    W[5, :] = np.float32(3e37) * np.sin(np.arange(64))
    for bits in (3, 4):
        for g in (0, 32):
            _compare(W, bits, g)


@pytest.mark.parametrize("bits", [3, 4])
def test_quotients_at_and_next_to_ties(bits):
    """Rows whose quotients w/s sit on half-integers or a few ulps beside them: the
    rounding decision must be the one of the correctly rounded binary32 division."""
    qmax = (1 << bits) - 1
    rng = np.random.default_rng(40 + bits)
    K = 512
    rows = []
    for step in (1.0, 0.5, 0.1, 0.3, 1e-3, 7.7, 3e-5, 1234.5):
        s = np.float32(step)
        k = rng.integers(0, qmax, size=K).astype(np.float32)
        x = ((k + np.float32(0.5)) * s).astype(np.float32)
        # walk up to 3 representable numbers to either side
        for _ in range(3):
            up = rng.integers(0, 3, size=K)
            toward = np.where(up == 1, np.float32(np.inf), np.float32(-np.inf)).astype(np.float32)
            x = np.where(up == 0, x, np.nextafter(x, toward)).astype(np.float32)
        for shift in (0.0, -2.0 * step, 3.0 * step):
            r = (x + np.float32(shift)).astype(np.float32)
            # pin the group's range so that s is `step` (up to rounding) in every 32-column group
            r[0::32] = np.float32(shift)
            r[1::32] = np.float32(shift) + np.float32(qmax) * s
            rows.append(r)
    W = np.stack(rows).astype(np.float32)
    for g in (0, 32, 128):
        _compare(W, bits, g)


def test_tiny_and_subnormal_scales():
    K = 256
    W = np.zeros((6, K), np.float32)
    j = np.arange(K, dtype=np.float64)
    W[0] = (1e-39 * j).astype(np.float32)                 # subnormal weights, subnormal scale
    W[1] = (1e-36 * np.sin(j)).astype(np.float32)         # 1/s beyond 1e30
    W[2] = (3e-31 * np.cos(j)).astype(np.float32)
    W[3] = np.float32(1000.0) + (1e-4 * (j % 7)).astype(np.float32)   # large |w/s|
    W[4] = np.float32(-5e4) + (2e-3 * (j % 5)).astype(np.float32)
    # the smallest range whose scale does not round to zero (below it Eq. 1 divides by 0)
    W[5, ::2] = np.float32(3e-44)
    for bits in (3, 4):
        for g in (0, 32):
            _compare(W, bits, g)


@pytest.mark.parametrize("K", [8192, 12288, 24576, 24704, 32768])
def test_row_lengths_across_the_register_budgets(K):
    d = synth.custom(K, 24, K, 1, 3, 128, outliers=True)
    _compare(d["W"], 3, 128)
    _compare(d["W"][:8], 4, 0)


@pytest.mark.parametrize("bits", [3, 4])
def test_pack_unpack_random_codes(bits):
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 1 << bits, size=(77, 1056), dtype=np.uint8)
    q = binding.pack(torch.from_numpy(codes).cuda(), bits)
    assert np.array_equal(u32(q), oracle.pack(codes, bits))
    raw = rng.integers(0, 2 ** 32, size=(77, 1056 * bits // 32), dtype=np.uint64).astype(np.uint32)
    c = binding.unpack(torch.from_numpy(raw.view(np.int32)).cuda(), 1056, bits)
    assert np.array_equal(c.cpu().numpy(), oracle.unpack(raw, 1056, bits))
    # codes with stray upper bits are masked
    dirty = codes | np.uint8(0xF0 if bits == 4 else 0xF8)
    q2 = binding.pack(torch.from_numpy(dirty).cuda(), bits)
    assert np.array_equal(u32(q2), u32(q))


def test_argument_errors():
    W = torch.zeros((4, 64), device="cuda")
    with pytest.raises(binding.PeqaError) as e:
        binding.quantize_rtn(W, 5)
    assert e.value.status == -2
    with pytest.raises(binding.PeqaError) as e:
        binding.quantize_rtn(W, 4, 48)
    assert e.value.status == -3
    with pytest.raises(binding.PeqaError) as e:
        binding.quantize_rtn(torch.zeros((4, 48), device="cuda"), 4)
    assert e.value.status == -3
