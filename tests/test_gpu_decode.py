"""GPU parity: the small-batch decode path (Sec. 3.1/3.3 matrix-vector regime) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def _check(d, bits, g, M, also_fwd=False):
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    K = d["W"].shape[1]
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    Xb = d["X"][:M]
    X = bf16_to_dev(Xb)
    # the output sits between two guard rows that must survive
    N = packed.shape[0]
    buf = torch.full((M + 2, N), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[1:M + 1]
    binding.qlinear_decode(qw, X, Y)
    binding.check_status()
    ref = oracle.fwd(Xb, packed, zeros, scales, bits, g)
    assert_close(dev_to_f64(Y), ref, f"decode M={M}")
    assert torch.all(buf[0] == 7.0) and torch.all(buf[M + 1] == 7.0)
    if also_fwd:
        Y2 = binding.qlinear_fwd(qw, X)
        binding.check_status()
        assert_close(dev_to_f64(Y), dev_to_f64(Y2), "decode vs fwd kernel")


@pytest.mark.parametrize("M", [1, 2, 4, 8, 9, 16])
@pytest.mark.parametrize("bits,g", [(3, 0), (4, 0), (3, 128), (4, 64), (3, 32)])
def test_small_shapes(M, bits, g):
    # N=200: ragged 128-row block; K=1408 = 2.75 steps of 512 columns
    d = synth.custom(7 * M + bits + g, 200, 1408, 16, bits, g, outliers=True)
    _check(d, bits, g, M, also_fwd=(M in (1, 16)))


def test_single_step_and_tiny_rows():
    d = synth.custom(2, 8, 128, 16, 3, 0)
    _check(d, 3, 0, 1)
    _check(d, 3, 0, 16)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_c4_llama65b_shapes(M):
    """Workload c4 (LLaMA-65B decode shapes) at full size: 3-bit per-channel, three layer shapes."""
    for d in synth.generate("c4"):
        _check(d, 3, 0, M)


@pytest.mark.parametrize("bits,g,M", [(3, 128, 1), (4, 128, 3), (3, 256, 2), (4, 0, 1), (3, 128, 9)])
def test_several_row_blocks_per_cta(bits, g, M):
    # N=5120 gives every CTA of the streaming kernel 40 rows (a full 32-row block and a
    # quarter of one); K=2048 is four 512-column steps, so warps beyond the fourth idle
    d = synth.custom(50 + bits + g + M, 5120, 2048, 16, bits, g, outliers=True)
    _check(d, bits, g, M)


def test_ring_reuse_with_long_rows():
    # 152 rows x 43 steps per CTA: the ring is refilled several times
    d = synth.custom(77, 22016 // 4, 22016 // 2, 2, 3, 128)
    _check(d, 3, 128, 1)


def test_unit_scale_integer_inputs_are_exact():
    rng = np.random.default_rng(0)
    N, K, M = 256, 1024, 5
    codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
    packed = oracle.pack(codes, 3)
    qw = to_qweight(packed, np.zeros((N, 1), np.uint8), np.ones((N, 1), np.float32), 3, 0, K)
    Xi = rng.integers(-4, 5, size=(M, K))
    Y = binding.qlinear_decode(qw, bf16_to_dev(synth.f32_to_bf16_bits(Xi.astype(np.float32))))
    ref = (Xi @ codes.astype(np.int64).T).astype(np.float32)
    exp = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(ref)).astype(np.float64)
    assert np.array_equal(dev_to_f64(Y), exp)


@pytest.mark.parametrize("bits,M", [(3, 1), (4, 5), (3, 16)])
def test_multitask_scales(bits, M):
    """Sec. 3.3: one frozen Q, z; token m is decoded with the scale vector of its own task."""
    N, K = 1032, 1024
    d = synth.custom(70 + bits + M, N, K, 16, bits, 0, outliers=True)
    codes, zeros, scales, packed = oracle_layer(d, bits, 0)
    rng = np.random.default_rng(M)
    table = (scales[:, 0][None, :] * rng.uniform(0.5, 2.0, size=(3, N))).astype(np.float32)
    ids = rng.integers(0, 3, size=M).astype(np.int32)
    qw = to_qweight(packed, zeros, scales, bits, 0, K)
    Xb = d["X"][:M]
    Y = binding.qlinear_decode_multitask(qw, torch.from_numpy(table).cuda(),
                                         torch.from_numpy(ids).cuda(), bf16_to_dev(Xb))
    torch.cuda.synchronize()
    binding.check_status()
    ref = oracle.fwd_multitask(Xb, packed, zeros, table, ids, bits)
    assert_close(dev_to_f64(Y), ref, "multi-task decode")
    # ids beyond the table are clamped to its last row
    Y2 = binding.qlinear_decode_multitask(qw, torch.from_numpy(table).cuda(),
                                          torch.from_numpy(np.where(ids == 2, 7, ids).astype(np.int32)).cuda(),
                                          bf16_to_dev(Xb))
    assert torch.equal(Y, Y2)


def test_multitask_rejects_grouped_layers():
    d = synth.custom(5, 64, 256, 16, 4, 128)
    codes, zeros, scales, packed = oracle_layer(d, 4, 128)
    qw = to_qweight(packed, zeros, scales, 4, 128, 256)
    with pytest.raises(binding.PeqaError):
        binding.qlinear_decode_multitask(qw, torch.ones((2, 64), device="cuda"),
                                         torch.zeros(1, dtype=torch.int32, device="cuda"),
                                         bf16_to_dev(d["X"][:1]))
