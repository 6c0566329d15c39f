"""GPU parity: forward, dX and dS of the PEQA layer (Eq. 2) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import (assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight)

pytestmark = pytest.mark.gpu


def _run_all(d, bits, g, check=("Y", "dX", "dS")):
    spec = d["spec"]
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    K = d["W"].shape[1]
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    X = bf16_to_dev(d["X"])
    dY = bf16_to_dev(d["dY"])
    out = {}
    T, N = X.shape[0], packed.shape[0]
    G = scales.shape[1]

    # every output sits between two guard rows that must survive (in place of a memory checker)
    def guarded(rows, cols, dtype):
        flat = torch.full((rows * cols + 512,), 7.0, dtype=dtype, device="cuda")
        return flat, flat[256:256 + rows * cols].view(rows, cols)

    guards = []
    if "Y" in check:
        gb, Y = guarded(T, N, torch.bfloat16)
        guards.append(gb)
        binding.qlinear_fwd(qw, X, Y)
        out["Y"] = assert_close(dev_to_f64(Y), oracle.fwd(d["X"], packed, zeros, scales, bits, g), "Y")
    dX = dS = None
    if "dX" in check:
        gb, dX = guarded(T, K, torch.bfloat16)
        guards.append(gb)
    if "dS" in check:
        gb, dS = guarded(N, G, torch.float32)
        guards.append(gb)
    dX, dS = binding.qlinear_bwd(qw, X, dY, dX=dX, dS=dS, need_dx="dX" in check, need_ds="dS" in check)
    binding.check_status()
    for gb in guards:
        assert torch.all(gb[:256] == 7.0) and torch.all(gb[-256:] == 7.0), "a kernel wrote outside its output"
    if "dX" in check:
        out["dX"] = assert_close(dev_to_f64(dX), oracle.bwd_dx(d["dY"], packed, zeros, scales, K, bits, g), "dX")
    if "dS" in check:
        out["dS"] = assert_close(dev_to_f64(dS), oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, g), "dS")
    return out


def test_c1_four_bit_per_channel():
    d = next(synth.generate("c1"))
    _run_all(d, 4, 0)


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 0), (3, 64), (4, 128), (3, 32), (4, 256), (3, 192)])
def test_ragged_multi_tile(bits, g):
    # N=328 (2.56 row tiles, multiple of 8), K=768 (3 column tiles of 256), T=300 (ragged token tile)
    d = synth.custom(100 + bits + g, 328, 768, 300, bits, g, outliers=True, sigma_dy=1e-2)
    _run_all(d, bits, g)


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 0), (3, 64), (4, 32), (3, 192)])
def test_in_features_not_a_multiple_of_128(bits, g):
    # K = 192 and 576 are multiples of 64 only: 3-bit rows then have no 16-byte pitch and the
    # kernels read the packed codes directly instead of through TMA
    for K in (192, 576):
        d = synth.custom(200 + bits + g + K, 264, K, 150, bits, g, outliers=True, sigma_dy=1e-2)
        _run_all(d, bits, g)


@pytest.mark.parametrize("g", [0, 64, 192])
def test_token_tail_beyond_one_block(g):
    # T = 530 leaves 18 tokens in the second 512-token tile; T = 300 fills a block and a bit
    for T, K in ((530, 192 if g == 192 else 320), (300, 384)):
        d = synth.custom(300 + g + T, 264, K, T, 4, g, outliers=True, sigma_dy=1e-2)
        _run_all(d, 4, g)


@pytest.mark.parametrize("bits,g,N,K,T", [(4, 0, 8, 64, 3), (3, 0, 8, 64, 1), (4, 32, 40, 128, 513),
                                          (3, 128, 24, 128, 9), (4, 64, 8, 4096, 2)])
def test_layers_smaller_than_one_tile(bits, g, N, K, T):
    # every TMA box is larger than the tensor it reads; 3-bit K=64 takes the single-CTA kernels
    d = synth.custom(500 + N + K + T, N, K, T, bits, g, outliers=True, sigma_dy=1e-2)
    _run_all(d, bits, g)


@pytest.mark.parametrize("T", [1, 7, 64, 257, 513])
def test_token_counts(T):
    d = synth.custom(T, 256, 512, T, 3, 128, sigma_dy=1e-2)
    _run_all(d, 3, 128)


@pytest.mark.parametrize("bits", [3, 4])
def test_unit_scale_integer_inputs_are_exact(bits):
    """s=1, z=0, small-integer activations: every fp32 partial sum is an exact integer."""
    rng = np.random.default_rng(bits)
    T, N, K = 200, 264, 640
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    packed = oracle.pack(codes, bits)
    zeros = np.zeros((N, 1), np.uint8)
    scales = np.ones((N, 1), np.float32)
    Xi = rng.integers(-4, 5, size=(T, K))
    dYi = rng.integers(-2, 3, size=(T, N))
    Xb = synth.f32_to_bf16_bits(Xi.astype(np.float32))
    dYb = synth.f32_to_bf16_bits(dYi.astype(np.float32))
    qw = to_qweight(packed, zeros, scales, bits, 0, K)
    Y = binding.qlinear_fwd(qw, bf16_to_dev(Xb))
    dX, dS = binding.qlinear_bwd(qw, bf16_to_dev(Xb), bf16_to_dev(dYb))
    binding.check_status()
    Yref = (Xi @ codes.astype(np.int64).T).astype(np.float32)
    Yexp = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(Yref)).astype(np.float64)
    assert np.array_equal(dev_to_f64(Y), Yexp)
    dXref = (dYi @ codes.astype(np.int64)).astype(np.float32)
    dXexp = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(dXref)).astype(np.float64)
    assert np.array_equal(dev_to_f64(dX), dXexp)
    dSref = ((dYi.T @ Xi) * codes.astype(np.int64)).sum(axis=1)
    assert np.array_equal(dev_to_f64(dS)[:, 0], dSref.astype(np.float64))


def test_results_are_deterministic():
    d = synth.custom(3, 512, 512, 384, 4, 0, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 512)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    a = [binding.qlinear_fwd(qw, X), *binding.qlinear_bwd(qw, X, dY)]
    b = [binding.qlinear_fwd(qw, X), *binding.qlinear_bwd(qw, X, dY)]
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_skipping_outputs_and_workspace_errors():
    d = synth.custom(4, 128, 512, 64, 4, 0)
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 512)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    dX, dS = binding.qlinear_bwd(qw, None, dY, need_ds=False)
    assert dS is None and dX is not None
    assert binding.workspace_bytes(binding.OP_BWD, 64, qw) == 128 * 4 * 4
    import ctypes
    cs = qw.c_struct()
    dSbuf = torch.empty((128, 1), device="cuda")
    st = binding.lib().peqa_qlinear_bwd(ctypes.byref(cs), X.data_ptr(), dY.data_ptr(), 64, 0,
                                        dSbuf.data_ptr(), 0, 0, 0)
    assert st == -5
    torch.cuda.synchronize()


def test_c2_llama7b_attention_projection_full():
    """Workload c2 (LLaMA-7B attention projection) at full size; the oracle finishes each tensor in seconds."""
    d = next(synth.generate("c2"))
    res = _run_all(d, 3, 128)
    print("c2 errors (rel-L2, max-abs):", res)


@pytest.mark.parametrize("bits,g,N,K", [(3, 128, 2560, 256), (4, 0, 256, 2560)])
def test_last_round_of_tiles_cut_in_halves(bits, g, N, K):
    """4096 tokens give 8 token tiles; with 10 tiles along the output (N = 2560 for the forward,
    K = 2560 for dX) that is 80 tiles for the 74 CTA pairs of a 148-SM part, so the six tiles of
    the last round run as twelve items of 256 tokens.  Every output element is checked."""
    d = synth.custom(17 + bits, N, K, 4096, bits, g, outliers=True, sigma_dy=1e-2)
    _run_all(d, bits, g, check=("Y", "dX"))
