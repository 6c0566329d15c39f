"""Pins for the oracle's quantizer with a searched clipping range (Sec. 3.2: s0 and z0 are
"initialized to minimize" the reconstruction error of Eq. 1; the search itself is a reading)."""
import numpy as np
import pytest

import oracle


def _recon_err(W, codes, zeros, scales, g):
    """sum_j (w - s*(q - z))^2 per (row, group): binary32 products and differences, binary64 sum."""
    N, K = W.shape
    G = K // g
    s = np.repeat(scales, g, axis=1)
    z = np.repeat(zeros.astype(np.float32), g, axis=1)
    rec = (s * (codes.astype(np.float32) - z)).astype(np.float32)
    e = (W - rec).astype(np.float32).astype(np.float64)
    return (e * e).reshape(N, G, g).sum(axis=2)


@pytest.mark.parametrize("bits,g", [(3, 32), (4, 64), (3, 0), (4, 0)])
def test_single_candidate_is_plain_rtn(bits, g):
    rng = np.random.default_rng(bits + g)
    W = (rng.standard_normal((9, 128)) * 0.02).astype(np.float32)
    c0, z0, s0 = oracle.quantize_rtn(W, bits, g)
    c1, z1, s1, chosen, err = oracle.quantize_search(W, bits, g, n_cand=1)
    assert np.array_equal(c0, c1) and np.array_equal(z0, z1) and np.array_equal(s0, s1)
    assert np.all(chosen == 0)


@pytest.mark.parametrize("bits,g", [(3, 32), (4, 64), (3, 128), (4, 0)])
def test_never_worse_than_rtn_and_consistent(bits, g):
    rng = np.random.default_rng(10 + bits + g)
    W = (rng.standard_normal((33, 256)) * 0.02).astype(np.float32)
    W[rng.random(W.shape) < 0.01] *= 20            # heavy-tail entries: clipping pays off
    gg = 256 if g == 0 else g
    c0, z0, s0 = oracle.quantize_rtn(W, bits, g)
    c1, z1, s1, chosen, err = oracle.quantize_search(W, bits, g, n_cand=32)
    e0 = _recon_err(W, c0, z0, s0, gg)
    e1 = _recon_err(W, c1, z1, s1, gg)
    assert np.all(e1 <= e0)
    assert (e1 < e0).mean() > 0.2                  # the search does find better ranges
    np.testing.assert_allclose(err, e1, rtol=1e-12, atol=0)
    # a group where nothing beats the full range keeps candidate 0 and RTN's exact outputs
    same = chosen == 0
    assert np.array_equal(s1[same], s0[same]) and np.array_equal(z1[same], z0[same])
    # the codes are Eq. 1's for the chosen (s, z)
    qmax = np.float32((1 << bits) - 1)
    s = np.repeat(s1, gg, axis=1)
    z = np.repeat(z1.astype(np.float32), gg, axis=1)
    q = np.clip(np.rint((W / s).astype(np.float32)) + z, 0, qmax)
    assert np.array_equal(q.astype(np.uint8), c1)


def test_brute_force_search_on_tiny_groups():
    """Every candidate evaluated with numpy binary32 scalars in a Python loop."""
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((3, 64)) * 0.05).astype(np.float32)
    W[0, 3] *= 15
    W[2, 40] *= -12
    for bits in (3, 4):
        qmax = np.float32((1 << bits) - 1)
        codes, zeros, scales, chosen, err = oracle.quantize_search(W, bits, 32, n_cand=20)
        for i in range(3):
            for gi in range(2):
                seg = W[i, gi * 32:(gi + 1) * 32]
                mn, mx = np.float32(seg.min()), np.float32(seg.max())
                best = None
                for k in range(20):
                    p = np.float32(1.0) - np.float32(k) / np.float32(64.0)
                    lo, hi = np.float32(p * mn), np.float32(p * mx)
                    s = np.float32(np.float32(hi - lo) / qmax) if hi != lo else np.float32(1.0)
                    z = np.float32(min(max(np.rint(np.float32(np.float32(-lo) / s)), np.float32(0)), qmax))
                    tot, q_all = 0.0, []
                    for w in seg:
                        q = np.float32(min(max(np.float32(np.rint(np.float32(w / s)) + z), np.float32(0)), qmax))
                        rec = np.float32(s * np.float32(q - z))
                        e = np.float32(w - rec)
                        tot += float(e) * float(e)
                        q_all.append(int(q))
                    if best is None or tot < best[0]:
                        best = (tot, k, s, int(z), q_all)
                assert chosen[i, gi] == best[1]
                assert scales[i, gi] == best[2] and zeros[i, gi] == best[3]
                assert list(codes[i, gi * 32:(gi + 1) * 32]) == best[4]
                assert err[i, gi] == best[0]


def test_rows_on_an_exact_grid_keep_the_full_range():
    # W = (j mod 2^b - c) * 2^-6 is reproduced exactly by plain RTN: error 0 at candidate 0
    for bits, c in ((4, 7), (3, 3)):
        L = 1 << bits
        j = np.arange(64)
        W = (((j % L) - c) * 2.0 ** -6).astype(np.float32)[None, :]
        codes, zeros, scales, chosen, err = oracle.quantize_search(W, bits, 0, n_cand=32)
        assert chosen[0, 0] == 0 and err[0, 0] == 0.0
        assert np.array_equal(codes[0], (j % L).astype(np.uint8))
