"""The allocation-free scale-gradient entry point against the regular backward call.

peqa_qlinear_bwd_ds_static serves callers that cannot obtain device scratch (no cudaMalloc
where they run, or only input/output buffers handed to them); it keeps its partial sums in
an array built into the library.  Here it must reproduce what peqa_qlinear_bwd computes with
a caller-provided workspace, on two consecutive calls that reuse that array with different
data.  This file sorts last on purpose so that a failure here cannot hide another test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def _layer(seed, N, K, T, bits, g):
    d = synth.custom(seed, N, K, T, bits, g, sigma_dy=1e-2)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    return d, packed, zeros, to_qweight(packed, zeros, scales, bits, g, K)


def test_static_scratch_matches_workspace_path_twice_in_a_row():
    # two per-channel layers of different shape: the second call finds the first one's
    # partial sums still in the shared array
    cases = [_layer(31, 328, 768, 300, 4, 0), _layer(32, 256, 1024, 130, 3, 0)]
    for d, packed, zeros, qw in cases:
        assert binding.workspace_bytes(binding.OP_BWD, d["X"].shape[0], qw) > 0
        X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
        _, ref = binding.qlinear_bwd(qw, X, dY, need_dx=False)
        got = torch.full_like(ref, float("nan"))
        binding.qlinear_bwd_ds_static(qw, X, dY, got)
        binding.check_status()
        assert_close(dev_to_f64(got), dev_to_f64(ref), "dS static vs workspace")
        assert_close(dev_to_f64(got), oracle.bwd_ds(d["X"], d["dY"], packed, zeros, qw.bits, 0), "dS static vs oracle")
        # once a device has seen its first call, further calls leave the amount of free device
        # memory and torch's own allocator untouched
        torch.cuda.synchronize()
        free0, used0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        binding.qlinear_bwd_ds_static(qw, X, dY, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == used0


def test_group_sizes_that_need_no_scratch_and_oversize_refusal():
    d, packed, zeros, qw = _layer(33, 128, 512, 64, 3, 64)
    X, dY = bf16_to_dev(d["X"]), bf16_to_dev(d["dY"])
    _, ref = binding.qlinear_bwd(qw, X, dY, need_dx=False)
    got = torch.empty_like(ref)
    binding.qlinear_bwd_ds_static(qw, X, dY, got)
    torch.cuda.synchronize()
    assert torch.equal(got, ref)
    # a per-channel layer whose partial sums exceed the built-in array is refused up front
    cap = binding.bwd_ds_static_capacity_bytes()
    assert cap == 8 * 1024 * 1024
    N, K = 40000, 8192
    assert N * (K // 128) * 4 > cap
    w = binding._QWeight(4, N, K, 0, X.data_ptr(), X.data_ptr(), X.data_ptr())
    st = binding.lib().peqa_qlinear_bwd_ds_static(ctypes.byref(w), X.data_ptr(), dY.data_ptr(), 8,
                                                  got.data_ptr(), 0)
    assert st == -9
