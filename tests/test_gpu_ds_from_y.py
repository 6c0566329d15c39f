"""GPU parity: per-channel dS from the stored forward output (Eq. 2 with one scale per channel)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("bits,N,K,T", [(4, 264, 192, 150), (3, 328, 768, 300), (4, 1032, 64, 2049),
                                        (3, 8, 128, 1)])
def test_matches_the_oracle_on_the_same_stored_output(bits, N, K, T):
    d = synth.custom(400 + bits + N + T, N, K, T, bits, 0, outliers=True, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, 0)
    qw = to_qweight(packed, zeros, scales, bits, 0, K)
    Y = binding.qlinear_fwd(qw, bf16_to_dev(d["X"]))
    dS = binding.qlinear_bwd_ds_from_y(qw, bf16_to_dev(d["dY"]), Y)
    torch.cuda.synchronize()
    binding.check_status()
    got = dS.cpu().numpy().astype(np.float64)
    # same inputs, fp32 against fp64 accumulation: tight
    ref = oracle.bwd_ds_from_y(d["dY"], _bits(Y), scales)
    assert np.linalg.norm(got - ref) <= 2e-5 * np.linalg.norm(ref)
    # against the definition of dS (through dY^T X): the bf16 rounding of Y is all that differs
    full = oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, 0)
    assert_close(got, full, "dS from stored Y")
    # and against the library's own contraction kernel
    dS2 = binding.qlinear_bwd(qw, bf16_to_dev(d["X"]), bf16_to_dev(d["dY"]), need_dx=False)[1]
    assert_close(got, dS2.cpu().numpy().astype(np.float64), "dS from stored Y vs dS kernel")


def test_c3_gate_projection_full_size():
    """Workload c3 (LLaMA-7B MLP, 4-bit per-channel) at full size, every channel."""
    d = next(synth.generate("c3"))
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    K = d["W"].shape[1]
    qw = to_qweight(packed, zeros, scales, 4, 0, K)
    Y = binding.qlinear_fwd(qw, bf16_to_dev(d["X"]))
    dS = binding.qlinear_bwd_ds_from_y(qw, bf16_to_dev(d["dY"]), Y)
    torch.cuda.synchronize()
    ref = oracle.bwd_ds_from_y(d["dY"], _bits(Y), scales)
    got = dS.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) <= 2e-5 * np.linalg.norm(ref)
    rows = np.arange(0, d["W"].shape[0], 97, dtype=np.int32)
    full = oracle.bwd_ds(d["X"], d["dY"], packed, zeros, 4, 0, rows=rows)
    assert_close(got[rows], full, "dS from stored Y, sampled rows")


def test_rejects_grouped_layers_and_short_workspace():
    d = synth.custom(3, 64, 256, 16, 4, 128)
    codes, zeros, scales, packed = oracle_layer(d, 4, 128)
    qw = to_qweight(packed, zeros, scales, 4, 128, 256)
    Y = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PeqaError):
        binding.qlinear_bwd_ds_from_y(qw, Y, Y)
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 256)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")[:16]
    with pytest.raises(binding.PeqaError):
        binding.qlinear_bwd_ds_from_y(qw, Y, Y, workspace=ws)
