"""The time-out path of the tensor-core kernels: a stage that never fills must end the kernel
through its bounded waits, report PEQA_ERR_DEVICE_TIMEOUT on the stream it ran on, and leave
the context usable.  Nothing here traps or spins without a bound: the forward kernel is told
to expect one byte more than its copies deliver and its waits are limited to a millisecond."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight

pytestmark = pytest.mark.gpu


def test_starved_forward_times_out_and_the_next_call_is_correct():
    d = next(synth.generate("c1"))
    spec = d["spec"]
    codes, zeros, scales, packed = oracle_layer(d, spec.bits, spec.group_size)
    qw = to_qweight(packed, zeros, scales, spec.bits, spec.group_size, spec.K)
    X = bf16_to_dev(d["X"])
    ref = oracle.fwd(d["X"], packed, zeros, scales, spec.bits, spec.group_size)

    Y = binding.qlinear_fwd(qw, X)
    binding.check_status()
    assert_close(dev_to_f64(Y), ref, "forward before the self-test")

    other = torch.cuda.Stream()
    binding.selftest_configure(wait_limit_us=1000, starve_forward=True)
    try:
        binding.qlinear_fwd(qw, X)
        torch.cuda.synchronize()                      # the kernel returns by itself
        # a stream that ran nothing reports nothing
        with torch.cuda.stream(other):
            binding.check_status()
        with pytest.raises(binding.PeqaError) as err:
            binding.check_status()
        assert err.value.status == -8                 # PEQA_ERR_DEVICE_TIMEOUT
        binding.check_status()                        # reading the status cleared it
    finally:
        binding.selftest_configure()                  # defaults back

    Y2 = binding.qlinear_fwd(qw, X)
    dX, dS = binding.qlinear_bwd(qw, X, bf16_to_dev(d["dY"]))
    binding.check_status()
    assert_close(dev_to_f64(Y2), ref, "forward after the time-out")
    assert torch.equal(Y, Y2)
    assert_close(dev_to_f64(dS), oracle.bwd_ds(d["X"], d["dY"], packed, zeros, spec.bits, spec.group_size),
                 "dS after the time-out")


def test_status_words_are_per_stream():
    d = synth.custom(3, 256, 256, 64, 4, 0)
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 256)
    X = bf16_to_dev(d["X"])
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    binding.selftest_configure(wait_limit_us=1000, starve_forward=True)
    try:
        with torch.cuda.stream(s1):
            binding.qlinear_fwd(qw, X)
        torch.cuda.synchronize()
        with torch.cuda.stream(s2):
            binding.check_status()                    # s2 ran nothing: clean
        with torch.cuda.stream(s1):
            with pytest.raises(binding.PeqaError):
                binding.check_status()
    finally:
        binding.selftest_configure()
    with torch.cuda.stream(s1):
        Y = binding.qlinear_fwd(qw, X)
        binding.check_status()
    ref = oracle.fwd(d["X"], packed, zeros, scales, 4, 0)
    assert_close(dev_to_f64(Y), ref, "forward on the stream that had timed out")
