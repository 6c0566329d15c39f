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
    """The documented layout written out with numpy.  Block (rg, t) = 8 rows x 512 columns (zero
    codes beyond K and in the row group that completes an odd count), blocks ordered
    (rg / 2, t, rg % 2); lane 4*r + c4 owns columns 8*c4..8*c4+7 of each of the 16 runs; string s =
    runs 4s..4s+3, string column cs = 8*(run % 4) + column % 8, stored at code position lo[cs/2]
    (cs even) or hi[cs/2] (cs odd); the lane's 4*bits words go out as chunks of four words,
    chunk-major within the block."""
    codes = oracle.unpack(packed, K, bits)
    N = codes.shape[0]
    T = -(-K // 512)
    N2 = -(-N // 16) * 16
    padded = np.zeros((N2, T * 512), np.uint8)
    padded[:N, :K] = codes
    N = N2
    lo, hi = _positions(bits)
    assert sorted(lo + hi) == list(range(32))
    pos = np.empty(32, int)
    pos[0::2], pos[1::2] = lo, hi
    v = padded.reshape(N // 8, 8, T, 4, 4, 4, 8)              # rg, r, t, s, run % 4, c4, e
    v = v.transpose(0, 2, 1, 5, 3, 4, 6)                      # rg, t, r, c4, s, run % 4, e
    strings = np.ascontiguousarray(v).reshape(-1, 32)         # string column cs = 8*(run % 4) + e
    placed = np.empty_like(strings)
    placed[:, pos] = strings
    words = oracle.pack(placed, bits)                         # [strings, bits] words
    lane_words = words.reshape(N // 16, 2, T, 32, bits, 4)    # rg / 2, rg % 2, t, lane, chunk c, word (wi = 4c + wo)
    out = np.ascontiguousarray(lane_words.transpose(0, 2, 1, 4, 3, 5))   # rg / 2, t, rg % 2, c, lane, word
    return out.reshape(-1)


@pytest.mark.parametrize("bits,N,K", [(3, 8, 128), (4, 8, 128), (3, 200, 1408), (4, 72, 640), (3, 1024, 4096),
                                      (4, 16, 512)])
def test_layout_and_inverse(bits, N, K):
    rng = np.random.default_rng(bits * 1000 + N + K)
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    packed = oracle.pack(codes, bits)
    qw = to_qweight(packed, np.zeros((N, 1), np.uint8), np.ones((N, 1), np.float32), bits, 0, K)
    assert binding.decode_prepared_bytes(qw) == (-(-N // 16) * 2) * (-(-K // 512)) * bits * 512
    prep = binding.decode_prepare(qw)
    torch.cuda.synchronize()
    assert np.array_equal(u32(prep), prepared_layout_by_hand(packed, bits, K))
    back = torch.full((N, K * bits // 32), -1, dtype=torch.int32, device="cuda")
    binding.decode_unprepare(qw, prep, out=back)
    torch.cuda.synchronize()
    assert np.array_equal(u32(back), packed)


def _check(d, bits, M, g=0):
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    N, K = d["W"].shape
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    prep = binding.decode_prepare(qw)
    torch.cuda.synchronize()
    Xb = d["X"][:M]
    X = bf16_to_dev(Xb)
    # the output sits between two guard rows that must survive
    buf = torch.full((M + 2, N), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[1:M + 1]
    binding.qlinear_decode_prepared(qw, prep, X, Y)
    binding.check_status()
    ref = oracle.fwd(Xb, packed, zeros, scales, bits, g)
    assert_close(dev_to_f64(Y), ref, f"prepared decode M={M} g={g}")
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


@pytest.mark.parametrize("g", [64, 128, 256, 512, 1024])
@pytest.mark.parametrize("bits,M", [(3, 1), (4, 3), (3, 8), (4, 16), (3, 13)])
def test_grouped_scales(bits, M, g):
    """Group-wise scales (Sec. 4.2): scale and zero-point come off the sum group by group."""
    d = synth.custom(11 * M + bits + g, 328, 2048, 16, bits, g, outliers=True)
    _check(d, bits, M, g)


@pytest.mark.parametrize("bits,N,K,M,g", [(3, 200, 1408, 2, 64), (4, 72, 640, 9, 128), (3, 40, 16384, 16, 256),
                                          (3, 264, 22016, 9, 64), (4, 64, 16384, 16, 2048)])
def test_grouped_scales_ragged_steps_and_chunks(bits, N, K, M, g):
    # 1408 and 640 columns end inside a step of 512; 16 tokens x 16384 columns are staged in chunks
    d = synth.custom(bits + N + M + g, N, K, 16, bits, g, outliers=True)
    _check(d, bits, M, g)


def test_c5_group64_layer_shapes():
    """The LLaMA-65B layer shapes with 3-bit codes in groups of 64 (workload c5), M = 1 and 4."""
    seen = set()
    for d in synth.generate("c5", T=16):
        if d["W"].shape in seen:
            continue
        seen.add(d["W"].shape)
        for M in (1, 4):
            _check(d, 3, M, 64)


def test_first_launch_after_prepare_on_reused_memory():
    """The weights of a freshly prepared buffer come out of L2 much faster than in steady state;
    a ring slot must not be refilled before every lane has read it.  Repeats prepare -> decode
    on buffers the allocator hands out again (down-projection shape of LLaMA-65B, groups of 64)."""
    d = synth.custom(3, 2048, 22016, 4, 3, 64, outliers=True)
    codes, zeros, scales, packed = oracle_layer(d, 3, 64)
    refs = {M: oracle.fwd(d["X"][:M], packed, zeros, scales, 3, 64) for M in (1, 4)}
    for rep in range(6):
        for M in (1, 4):
            qw = to_qweight(packed, zeros, scales, 3, 64, 22016)
            prep = binding.decode_prepare(qw)
            torch.cuda.synchronize()
            Y = binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(d["X"][:M]))
            binding.check_status()
            assert_close(dev_to_f64(Y), refs[M], f"first launch after prepare, rep {rep}, M={M}")
            del qw, prep, Y


@pytest.mark.parametrize("bits,M,g", [(3, 1, 64), (4, 5, 128), (3, 16, 256), (4, 7, 512)])
def test_multitask_grouped_scales(bits, M, g):
    """Sec. 3.3 with group-wise scales: the task table is [n_tasks, N, G]."""
    N, K = 520, 1024
    d = synth.custom(170 + bits + M + g, N, K, 16, bits, g, outliers=True)
    codes, zeros, scales, packed = oracle_layer(d, bits, g)
    rng = np.random.default_rng(M + g)
    table = (scales[None] * rng.uniform(0.5, 2.0, size=(3, N, K // g))).astype(np.float32)
    ids = rng.integers(0, 3, size=M).astype(np.int32)
    qw = to_qweight(packed, zeros, scales, bits, g, K)
    prep = binding.decode_prepare(qw)
    tab = torch.from_numpy(table).cuda()
    torch.cuda.synchronize()
    Xb = d["X"][:M]
    Y = binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(Xb), scale_table=tab,
                                        task_ids=torch.from_numpy(ids).cuda())
    binding.check_status()
    ref = oracle.fwd_multitask(Xb, packed, zeros, table, ids, bits, g)
    assert_close(dev_to_f64(Y), ref, "multi-task grouped prepared decode")


def test_rejects_unsupported_groups_and_bad_shapes():
    d = synth.custom(5, 64, 256, 16, 4, 32)
    codes, zeros, scales, packed = oracle_layer(d, 4, 32)
    qw = to_qweight(packed, zeros, scales, 4, 32, 256)
    prep = binding.decode_prepare(qw)          # the layout does not depend on the groups
    with pytest.raises(binding.PeqaError):     # groups of 32 columns are served by qlinear_decode
        binding.qlinear_decode_prepared(qw, prep, bf16_to_dev(d["X"][:1]))
    d = synth.custom(6, 64, 96, 16, 4, 0)      # K % 128 != 0
    codes, zeros, scales, packed = oracle_layer(d, 4, 0)
    qw = to_qweight(packed, zeros, scales, 4, 0, 96)
    assert binding.decode_prepared_bytes(qw) == 0
