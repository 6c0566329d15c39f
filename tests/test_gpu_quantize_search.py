"""GPU parity (bit-exact): the quantizer with a searched clipping range against the oracle
(Sec. 3.2's error-minimising initialisation of s0, z0; Eq. 1 evaluated per candidate range)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import u32

pytestmark = pytest.mark.gpu


def _check(W, bits, g, n_cand):
    codes, zeros, scales, chosen, err = oracle.quantize_search(W, bits, g, n_cand)
    qw, ch = binding.quantize_search(torch.from_numpy(W).cuda(), bits, g, n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(ch.cpu().numpy(), chosen)
    assert np.array_equal(qw.scales.cpu().numpy(), scales)
    assert np.array_equal(qw.zeros.cpu().numpy(), zeros)
    assert np.array_equal(u32(qw.qweight), oracle.pack(codes, bits))
    return chosen


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("g,n_cand", [(32, 32), (64, 20), (128, 64), (0, 32), (0, 1)])
def test_matches_oracle_bit_for_bit(bits, g, n_cand):
    rng = np.random.default_rng(bits * 100 + g + n_cand)
    W = (rng.standard_normal((77, 512)) * 0.02).astype(np.float32)
    W[rng.random(W.shape) < 0.01] *= 20
    W[5, :32] = 0.25                       # a constant group (s := 1)
    W[6, :64] = np.abs(W[6, :64])          # a one-sided group (clamped z)
    chosen = _check(W, bits, g, n_cand)
    if n_cand > 1:
        assert (chosen > 0).any()


def test_llama_shaped_layers():
    d = next(synth.generate("c2"))
    _check(d["W"][:512], 3, 128, 32)
    d = next(synth.generate("c5"))
    _check(d["W"][:256], 3, 64, 32)


def test_single_candidate_equals_rtn_entry_point():
    rng = np.random.default_rng(1)
    W = (rng.standard_normal((64, 1024)) * 0.02).astype(np.float32)
    Wd = torch.from_numpy(W).cuda()
    a = binding.quantize_rtn(Wd, 3, 128)
    b, _ = binding.quantize_search(Wd, 3, 128, 1)
    torch.cuda.synchronize()
    assert torch.equal(a.qweight, b.qweight) and torch.equal(a.zeros, b.zeros) and torch.equal(a.scales, b.scales)
