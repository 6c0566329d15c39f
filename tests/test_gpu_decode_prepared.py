"""GPU parity of the decode path that reads a prepared copy of the frozen weights
(Sec. 3.1 / 3.3): the layout itself, its inverse, and the kernel against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_14152_b200 import binding, synth
from gpu_util import assert_close, bf16_to_dev, dev_to_f64, oracle_layer, to_qweight, u32

pytestmark = pytest.mark.gpu

# code positions inside a 32-column run, as the header documents them
LO3 = [1, 0, 3, 2, 4, 9, 12, 11, 15, 14, 18, 21, 24, 23, 26, 25]
HI3 = [5, 6, 7, 8, 10, 13, 16, 17, 19, 20, 22, 27, 28, 29, 30, 31]


def _positions(bits):
    if bits == 3:
        return LO3, HI3
    lo = [8 * (k // 4) + k % 4 for k in range(16)]
    return lo, [p + 4 for p in lo]


def prepared_layout_by_hand(packed, bits, K):
    """The documented layout written out with numpy: permute the codes of every 32-column run,
    pack them canonically, then move 16-byte chunks to ((rg*C + c)*U + u)*8 + r."""
    codes = oracle.unpack(packed, K, bits)
    N = codes.shape[0]
    lo, hi = _positions(bits)
    assert sorted(lo + hi) == list(range(32))
    perm = np.empty_like(codes).reshape(N, K // 32, 32)
    src = codes.reshape(N, K // 32, 32)
    for k in range(16):
        perm[:, :, lo[k]] = src[:, :, 2 * k]
        perm[:, :, hi[k]] = src[:, :, 2 * k + 1]
    words = oracle.pack(perm.reshape(N, K), bits)             # [N, K*bits/32]
    U, C = K // 128, bits
    units = words.reshape(N // 8, 8, U, C, 4)                 # rg, r, u, c, word
    out = np.ascontiguousarray(units.transpose(0, 3, 2, 1, 4))  # rg, c, u, r, word
    return out.reshape(-1)


@pytest.mark.parametrize("bits,N,K", [(3, 8, 128), (4, 8, 128), (3, 200, 1408), (4, 72, 640), (3, 1024, 4096)])
def test_layout_and_inverse(bits, N, K):
    rng = np.random.default_rng(bits * 1000 + N + K)
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    packed = oracle.pack(codes, bits)
    qw = to_qweight(packed, np.zeros((N, 1), np.uint8), np.ones((N, 1), np.float32), bits, 0, K)
    assert binding.decode_prepared_bytes(qw) == N * K * bits // 8
    prep = binding.decode_prepare(qw)
    torch.cuda.synchronize()
    assert np.array_equal(u32(prep), prepared_layout_by_hand(packed, bits, K))
    back = binding.decode_unprepare(qw, prep)
    torch.cuda.synchronize()
    assert np.array_equal(u32(back), packed)


def _check(d, bits, M, canary=True):
    codes, zeros, scales, packed = oracle_layer(d, bits, 0)
    N, K = d["W"].shape
    qw = to_qweight(packed, zeros, scales, bits, 0, K)
    prep = binding.decode_prepare(qw)
    torch.cuda.synchronize()
    Xb = d["X"][:M]
    X = bf16_to_dev(Xb)
    # the output sits between two guard rows that must survive
    buf = torch.full((M + 2, N), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[1:M + 1]
    binding.qlinear_decode_prepared(qw, prep, X, Y)
    binding.check_status()
    ref = oracle.fwd(Xb, packed, zeros, scales, bits, 0)
    assert_close(dev_to_f64(Y), ref, f"prepared decode M={M}")
    assert torch.all(buf[0] == 7.0) and torch.all(buf[M + 1] == 7.0)
    return qw, prep, X, Y


@pytest.mark.parametrize("M", [1, 2, 4, 8, 9, 16])
@pytest.mark.parametrize("bits", [3, 4])
def test_small_shapes(M, bits):
    # 200 rows = 25 row groups (CTAs with one group: half pairs); 1408 columns = 11 units
    d = synth.custom(7 * M + bits, 200, 1408, 16, bits, 0, outliers=True)
    _check(d, bits, M)


@pytest.mark.parametrize("bits,N,K,M", [(3, 8, 128, 1), (3, 8, 128, 16), (4, 16, 256, 3),
                                        (3, 5120, 2048, 5), (4, 2400, 1024, 12), (3, 1184, 512, 7)])
def test_pairs_rounds_and_ragged_groups(bits, N, K, M):
    # 5120 rows: 640 groups over the SMs give 5 groups per CTA (three pairs, the last half);
    # 2400 rows: 300 groups, 3 per CTA in all but the last CTA; 1184 rows: one group per CTA
    d = synth.custom(bits + N + K + M, N, K, 16, bits, 0, outliers=True)
    _check(d, bits, M)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_c4_llama65b_shapes(M):
    """Workload c4 (LLaMA-65B decode shapes) at full size: 3-bit per-channel, three layer shapes.
    M = 16 stages the activations in chunks of K."""
    for d in synth.generate("c4"):
        _check(d, 3, M)


def test_activations_staged_in_chunks():
    # 16 tokens x 16384 columns do not fit shared memory at once
    d = synth.custom(91, 64, 16384, 16, 4, 0)
    _check(d, 4, 16)
    d = synth.custom(92, 264, 22016, 16, 3, 0)
    _check(d, 3, 9)


def test_matches_canonical_decode_and_is_deterministic():
    d = synth.custom(12, 1024, 4096, 16, 3, 0, outliers=True)
    qw, prep, X, Y = _check(d, 3, 4)
    Yc = binding.qlinear_decode(qw, X)
    assert_close(dev_to_f64(Y), dev_to_f64(Yc), "prepared vs canonical decode")
    Y2 = binding.qlinear_decode_prepared(qw, prep, X)
    Y3 = binding.qlinear_decode_prepared(qw, prep, X)
    torch.cuda.synchronize()
    assert torch.equal(Y2, Y3) and torch.equal(Y2, Y)


def test_unit_scale_integer_inputs_are_exact():
    rng = np.random.default_rng(0)
    N, K, M = 256, 1024, 5
    for bits in (3, 4):
        codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
        packed = oracle.pack(codes, bits)
        qw = to_qweight(packed, np.zeros((N, 1), np.uint8), np.ones((N, 1), np.float32), bits, 0, K)
        prep = binding.decode_prepare(qw)
        torch.cuda.synchronize()
        Xi = rng.integers(-4, 5, size=(M, K))
        Y = binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(synth.f32_to_bf16_bits(Xi.astype(np.float32))))
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
    prep = binding.decode_prepare(qw)
    tab = torch.from_numpy(table).cuda()
    torch.cuda.synchronize()
    Xb = d["X"][:M]
    Y = binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(Xb), scale_table=tab,
                                        task_ids=torch.from_numpy(ids).cuda())
    binding.check_status()
    ref = oracle.fwd_multitask(Xb, packed, zeros, table, ids, bits)
    assert_close(dev_to_f64(Y), ref, "multi-task prepared decode")


def test_rejects_grouped_layers_and_bad_shapes():
    d = synth.custom(5, 64, 256, 16, 4, 128)
    codes, zeros, scales, packed = oracle_layer(d, 4, 128)
    qw = to_qweight(packed, zeros, scales, 4, 128, 256)
    prep = binding.decode_prepare(qw)          # the layout does not depend on the groups
    with pytest.raises(binding.PeqaError):
        binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(d["X"][:1]))
    d = synth.custom(6, 64, 96, 16, 4, 0)      # K % 128 != 0
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 96)
    assert binding.decode_prepared_bytes(qw) == 0
