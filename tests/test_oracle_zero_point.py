"""Pins for the oracle's layer with a real-valued zero-point (App. K trains z as well as s;
the weight is still Eq. 2's s * (Q - z), with z off the integer grid)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2305_14152_b200 import synth


def _case(seed, N, K, T, bits, g, sigma_dy=1.0):
    d = synth.custom(seed, N, K, T, bits, g, sigma_dy=sigma_dy)
    codes, zeros, scales = oracle.quantize_rtn(d["W"], bits, g)
    rng = np.random.default_rng(seed)
    # a trained zero-point: the stored integer moved by a fraction, sometimes past the code range
    zf = (zeros.astype(np.float32) + rng.uniform(-1.3, 1.3, size=zeros.shape).astype(np.float32))
    return d, codes, zeros, zf, scales, oracle.pack(codes, bits)


def _f(bits16):
    return synth.bf16_bits_to_f32(bits16).astype(np.float64)


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32), (3, 0), (4, 64)])
def test_integral_zero_point_reduces_to_the_integer_functions(bits, g):
    d, codes, zeros, zf, scales, qw = _case(21, 24, 128, 9, bits, g)
    zi = zeros.astype(np.float32)
    assert np.array_equal(oracle.fwd_zf(d["X"], qw, zi, scales, bits, g), oracle.fwd(d["X"], qw, zeros, scales, bits, g))
    assert np.array_equal(oracle.bwd_dx_zf(d["dY"], qw, zi, scales, 128, bits, g),
                          oracle.bwd_dx(d["dY"], qw, zeros, scales, 128, bits, g))
    assert np.array_equal(oracle.bwd_ds_zf(d["X"], d["dY"], qw, zi, bits, g),
                          oracle.bwd_ds(d["X"], d["dY"], qw, zeros, bits, g))


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32)])
def test_brute_force_rational_arithmetic(bits, g):
    T, N, K = 3, 4, 64
    d, codes, zeros, zf, scales, qw = _case(22, N, K, T, bits, g)
    gg = K if g == 0 else g
    X = synth.bf16_bits_to_f32(d["X"])
    dY = synth.bf16_bits_to_f32(d["dY"])
    Wbar = [[int(codes[i, j]) - Fraction(float(zf[i, j // gg])) for j in range(K)] for i in range(N)]
    Wh = [[Fraction(float(scales[i, j // gg])) * Wbar[i][j] for j in range(K)] for i in range(N)]
    Y = oracle.fwd_zf(d["X"], qw, zf, scales, bits, g)
    dX = oracle.bwd_dx_zf(d["dY"], qw, zf, scales, K, bits, g)
    dS = oracle.bwd_ds_zf(d["X"], d["dY"], qw, zf, bits, g)
    for t in range(T):
        for i in range(N):
            ref = sum(Fraction(float(X[t, j])) * Wh[i][j] for j in range(K))
            assert abs(Y[t, i] - float(ref)) <= 1e-12 * max(1.0, abs(float(ref)))
        for j in range(K):
            ref = sum(Fraction(float(dY[t, i])) * Wh[i][j] for i in range(N))
            assert abs(dX[t, j] - float(ref)) <= 1e-12 * max(1.0, abs(float(ref)))
    for i in range(N):
        for gi in range(K // gg):
            ref = Fraction(0)
            for j in range(gi * gg, (gi + 1) * gg):
                dw = sum(Fraction(float(dY[t, i])) * Fraction(float(X[t, j])) for t in range(T))
                ref += Wbar[i][j] * dw
            assert abs(dS[i, gi] - float(ref)) <= 1e-12 * max(1.0, abs(float(ref)))


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32)])
def test_gradients_are_finite_differences_of_the_affine_loss(bits, g):
    """L(s, z) = <dY, Y(s, z)> is affine in s and in z separately, so a step of any size in one
    scale or one zero-point changes L by exactly step * gradient."""
    d, codes, zeros, zf, scales, qw = _case(23, 12, 64, 7, bits, g)
    dY = _f(d["dY"])
    dS = oracle.bwd_ds_zf(d["X"], d["dY"], qw, zf, bits, g)
    dZ = oracle.bwd_dz(d["X"], d["dY"], scales, g)
    base = float((dY * oracle.fwd_zf(d["X"], qw, zf, scales, bits, g)).sum())
    for i in (0, 5, 11):
        for gi in range(scales.shape[1]):
            s2 = scales.copy()
            s2[i, gi] += np.float32(0.5)
            step = float(s2[i, gi]) - float(scales[i, gi])
            L = float((dY * oracle.fwd_zf(d["X"], qw, zf, s2, bits, g)).sum())
            assert abs((L - base) / step - dS[i, gi]) <= 1e-9 * max(1.0, abs(dS[i, gi]))
            z2 = zf.copy()
            z2[i, gi] += np.float32(0.75)
            step = float(z2[i, gi]) - float(zf[i, gi])
            L = float((dY * oracle.fwd_zf(d["X"], qw, z2, scales, bits, g)).sum())
            assert abs((L - base) / step - dZ[i, gi]) <= 1e-9 * max(1.0, abs(dZ[i, gi]))


def test_adjoint_identity_and_dense_matmul():
    bits, g = 3, 64
    d, codes, zeros, zf, scales, qw = _case(24, 40, 256, 33, bits, g, sigma_dy=1e-2)
    X, dY = _f(d["X"]), _f(d["dY"])
    Y = oracle.fwd_zf(d["X"], qw, zf, scales, bits, g)
    dX = oracle.bwd_dx_zf(d["dY"], qw, zf, scales, 256, bits, g)
    assert abs((dY * Y).sum() - (dX * X).sum()) <= 1e-10 * abs((dY * Y).sum())
    What = np.repeat(scales.astype(np.float64), g, axis=1) * \
        (codes.astype(np.float64) - np.repeat(zf.astype(np.float64), g, axis=1))
    np.testing.assert_allclose(Y, X @ What.T, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(dX, dY @ What, rtol=1e-11, atol=1e-14)
    # token and row selections pick the same values
    tok = np.array([0, 7, 32], np.int32)
    assert np.array_equal(oracle.fwd_zf(d["X"], qw, zf, scales, bits, g, tokens=tok), Y[tok])
    rows = np.array([1, 39], np.int32)
    assert np.array_equal(oracle.bwd_ds_zf(d["X"], d["dY"], qw, zf, bits, g, rows=rows),
                          oracle.bwd_ds_zf(d["X"], d["dY"], qw, zf, bits, g)[rows])
