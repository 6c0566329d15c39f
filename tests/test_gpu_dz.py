"""GPU parity: scale gradient and zero-point gradient (App. K) from the same dW tiles."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 0), (3, 64), (4, 128), (3, 32), (4, 256), (3, 192)])
def test_ragged_multi_tile(bits, g):
    # N=328 (2.56 row tiles), K=768 (3 column tiles of 256), T=300 (ragged token stages)
    d = synth.custom(600 + bits + g, 328, 768, 300, bits, g, outliers=True, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    qw = to_qweight(packed, zeros, scales, bits, g, 768)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    dS, dZ = binding.qlinear_bwd_dsdz(qw, X, dY)
    torch.cuda.synchronize()
    binding.check_status()
    assert_close(dS.cpu().numpy().astype(np.float64), oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, g), "dS")
    assert_close(dZ.cpu().numpy().astype(np.float64), oracle.bwd_dz(d["X"], d["dY"], scales, g), "dZ")
    # dS must not depend on whether dZ is asked for
    dS_only = binding.qlinear_bwd(qw, X, dY, need_dx=False)[1]
    assert torch.equal(dS, dS_only)


def test_c2_full_size():
    d = next(synth.generate("c2"))
    codes, zeros, scales, packed = oracle_layer(d, 3, 128)
    qw = to_qweight(packed, zeros, scales, 3, 128, d["W"].shape[1])
    dS, dZ = binding.qlinear_bwd_dsdz(qw, bf16_to_dev(d["X"]), bf16_to_dev(d["dY"]))
    torch.cuda.synchronize()
    rows = np.arange(0, d["W"].shape[0], 61, dtype=np.int32)
    assert_close(dZ.cpu().numpy().astype(np.float64)[rows], oracle.bwd_dz(d["X"], d["dY"], scales, 128, rows=rows), "dZ")
    assert_close(dS.cpu().numpy().astype(np.float64)[rows],
                 oracle.bwd_ds(d["X"], d["dY"], packed, zeros, 3, 128, rows=rows), "dS")
