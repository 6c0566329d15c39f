"""Pins for the oracle's RTN quantizer (paper Eq. 1, Sec. 3.2; group-wise variant Sec. 4.2)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(os.path.join(GOLD, path)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


def test_eq1_worked_examples_exact():
    for line in _rows("eq1_worked_examples.txt"):
        bits, c, scale, zero = line.split()
        bits, c, zero, scale = int(bits), int(c), int(zero), float(scale)
        L = 1 << bits
        j = np.arange(64)
        W = (((j % L) - c) * 2.0 ** -6).astype(np.float32)[None, :]
        codes, zeros, scales = oracle.quantize_rtn(W, bits)
        assert scales[0, 0] == np.float32(scale)
        assert zeros[0, 0] == zero
        assert np.array_equal(codes[0], (j % L).astype(np.uint8))
        # reconstruction is exact for these rows
        assert np.array_equal(scales[0, 0] * (codes[0].astype(np.float32) - zeros[0, 0]), W[0])


def test_eq1_exact_ties_round_half_to_even():
    """Rows whose quotients are exactly k + 1/2: the expected codes are literal hand values."""
    n = 0
    for line in _rows("eq1_tie_rows.txt"):
        bits, zero, h, exp = [part.strip() for part in line.split(";")]
        bits, zero = int(bits), int(zero)
        h = np.array([float(x) for x in h.split()], dtype=np.float64)
        exp = np.array([int(x) for x in exp.split()], dtype=np.uint8)
        W = (h * 2.0 ** -4).astype(np.float32)[None, :]
        assert np.array_equal(W.astype(np.float64)[0], h * 2.0 ** -4)      # exactly representable
        codes, zeros, scales = oracle.quantize_rtn(W, bits)
        assert scales[0, 0] == np.float32(2.0 ** -4)
        assert zeros[0, 0] == zero
        assert np.array_equal(codes[0], exp)
        # the same row as two groups of 16 columns is not defined (groups are multiples of 32);
        # as one group of a wider row it must give the same codes
        W2 = np.concatenate([W, W], axis=1)
        c2, z2, s2 = oracle.quantize_rtn(W2, bits, 32)
        assert np.array_equal(c2[0, :32], exp) and np.array_equal(c2[0, 32:], exp)
        n += 1
    assert n >= 4


def _numpy_rtn(W, bits, g):
    """Independent restatement with numpy binary32 array ops (IEEE, ties-to-even rint)."""
    N, K = W.shape
    qmax = np.float32((1 << bits) - 1)
    Wg = W.reshape(N, K // g, g)
    mn = Wg.min(axis=2)
    mx = Wg.max(axis=2)
    s = ((mx - mn) / qmax).astype(np.float32)
    s = np.where(mx == mn, np.float32(1.0), s)
    z = np.clip(np.rint((-mn) / s), 0, qmax).astype(np.float32)
    q = np.clip(np.rint(Wg / s[:, :, None]) + z[:, :, None], 0, qmax)
    return q.reshape(N, K).astype(np.uint8), z.astype(np.uint8), s


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("g", [0, 32, 64, 128])
def test_matches_numpy_binary32_restatement(bits, g):
    rng = np.random.default_rng(7 + bits + g)
    W = (rng.standard_normal((37, 256)) * 0.02).astype(np.float32)
    W[3, 5] *= 20
    codes, zeros, scales = oracle.quantize_rtn(W, bits, g)
    gg = 256 if g == 0 else g
    q2, z2, s2 = _numpy_rtn(W, bits, gg)
    assert np.array_equal(scales, s2)
    assert np.array_equal(zeros, z2)
    assert np.array_equal(codes, q2)


def test_scalar_brute_force_4x64():
    """A literal per-element loop in Python using numpy.float32 scalars."""
    rng = np.random.default_rng(11)
    W = (rng.standard_normal((4, 64)) * 0.05).astype(np.float32)
    for bits in (3, 4):
        codes, zeros, scales = oracle.quantize_rtn(W, bits, 32)
        qmax = np.float32((1 << bits) - 1)
        for i in range(4):
            for gi in range(2):
                seg = W[i, gi * 32:(gi + 1) * 32]
                mn, mx = np.float32(min(seg)), np.float32(max(seg))
                s = np.float32(np.float32(mx - mn) / qmax)
                z = np.float32(min(max(np.rint(np.float32(-mn) / s), np.float32(0)), qmax))
                assert scales[i, gi] == s and zeros[i, gi] == int(z)
                for j in range(32):
                    q = np.rint(np.float32(seg[j] / s)) + z
                    q = min(max(q, np.float32(0)), qmax)
                    assert codes[i, gi * 32 + j] == int(q)


@pytest.mark.parametrize("bits", [3, 4])
def test_invariants_random(bits):
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((64, 512)) * 0.02).astype(np.float32)
    qmax = (1 << bits) - 1
    for g in (0, 64):
        codes, zeros, scales = oracle.quantize_rtn(W, bits, g)
        gg = 512 if g == 0 else g
        assert codes.max() <= qmax
        cg = codes.reshape(64, 512 // gg, gg)
        # groups straddle zero here, so the minimum maps to code 0 and the maximum to >= qmax-1
        assert np.all(cg.min(axis=2) == 0)
        assert np.all(cg.max(axis=2) >= qmax - 1)
        # half-step reconstruction bound of a uniform quantizer (z not clamped for these groups)
        s = np.repeat(scales.astype(np.float64), gg, axis=1)
        z = np.repeat(zeros.astype(np.float64), gg, axis=1)
        err = np.abs(W.astype(np.float64) - s * (codes.astype(np.float64) - z))
        assert np.all(err <= s * (0.5 + 2.0 ** -16))


def test_group_equal_K_is_per_channel():
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((16, 128)) * 0.02).astype(np.float32)
    a = oracle.quantize_rtn(W, 3, 0)
    b = oracle.quantize_rtn(W, 3, 128)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_groups_are_independent_column_runs():
    """Quantizing a column slice on its own equals that group's part of the group-wise result."""
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((8, 256)) * 0.02).astype(np.float32)
    codes, zeros, scales = oracle.quantize_rtn(W, 4, 64)
    for gi in range(4):
        c, z, s = oracle.quantize_rtn(W[:, gi * 64:(gi + 1) * 64].copy(), 4, 0)
        assert np.array_equal(c, codes[:, gi * 64:(gi + 1) * 64])
        assert np.array_equal(z[:, 0], zeros[:, gi])
        assert np.array_equal(s[:, 0], scales[:, gi])


def test_degenerate_and_one_sided_rows():
    W = np.zeros((3, 64), np.float32)
    W[0, :] = 0.25                               # constant row: s := 1, all codes equal
    W[1, :] = np.linspace(1.0, 2.0, 64)          # all positive: z clamps to 0, low codes unused
    W[2, :] = -np.linspace(1.0, 2.0, 64)         # all negative: z clamps to qmax
    codes, zeros, scales = oracle.quantize_rtn(W, 4)
    assert scales[0, 0] == 1.0 and zeros[0, 0] == 0 and np.all(codes[0] == 0)
    assert zeros[1, 0] == 0 and codes[1].max() == 15 and codes[1].min() == 15
    assert zeros[2, 0] == 15 and codes[2].max() == 0
    # negative zero minimum
    W2 = np.zeros((1, 32), np.float32)
    W2[0, 1:] = np.arange(1, 32, dtype=np.float32)
    W2[0, 0] = -0.0
    c, z, s = oracle.quantize_rtn(W2, 3)
    assert z[0, 0] == 0 and c[0, 0] == 0 and c[0, -1] == 7


def test_binary64_quotients_change_only_rare_near_ties():
    rng = np.random.default_rng(21)
    W = (rng.standard_normal((256, 1024)) * 0.02).astype(np.float32)
    c32, z32, _ = oracle.quantize_rtn(W, 4, 128)
    c64, z64, _ = oracle.quantize_rtn_f64(W, 4, 128)
    diff = np.count_nonzero(c32 != c64)
    assert diff <= 1e-4 * W.size
    assert np.abs(c32.astype(int) - c64.astype(int)).max() <= 1


def test_table4_learnable_parameter_counts():
    """Per-channel PEQA trains one scale per output row of every linear in the decoder stack."""
    dims = {"llama-7b": (4096, 11008, 32), "llama-13b": (5120, 13824, 40),
            "llama-30b": (6656, 17920, 60), "llama-65b": (8192, 22016, 80)}
    for line in _rows("table4_learnable_params.txt"):
        model, printed = line.split()
        d, ffn, layers = dims[model]
        shapes = [(d, d)] * 4 + [(ffn, d)] * 2 + [(d, ffn)]
        n_scales = 0
        for (N, K) in shapes:
            W = np.zeros((1, K), np.float32)     # one row is enough to read G off the oracle
            n_scales += N * oracle.quantize_rtn(W, 4)[2].shape[1]
        assert round(n_scales * layers / 1e6, 2) == float(printed)
