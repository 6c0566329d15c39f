"""Pins for the oracle's forward, dX and dS (the layer built on the paper's Eq. 2, Sec. 3.2)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2305_14152_b200 import synth


def _case(seed, N, K, T, bits, g, sigma_dy=1.0):
    d = synth.custom(seed, N, K, T, bits, g, sigma_dy=sigma_dy)
    codes, zeros, scales = oracle.quantize_rtn(d["W"], bits, g)
    return d, codes, zeros, scales, oracle.pack(codes, bits)


def _f(bits16):
    return synth.bf16_bits_to_f32(bits16).astype(np.float64)


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32), (3, 0), (4, 64)])
def test_brute_force_rational_arithmetic(bits, g):
    """Literal triple loops in exact rational arithmetic on a tiny layer."""
    T, N, K = 3, 4, 64
    d, codes, zeros, scales, qw = _case(1, N, K, T, bits, g)
    gg = K if g == 0 else g
    X = synth.bf16_bits_to_f32(d["X"])
    dY = synth.bf16_bits_to_f32(d["dY"])
    Wh = [[Fraction(float(scales[i, j // gg])) * (int(codes[i, j]) - int(zeros[i, j // gg]))
           for j in range(K)] for i in range(N)]
    Y = oracle.fwd(d["X"], qw, zeros, scales, bits, g)
    dX = oracle.bwd_dx(d["dY"], qw, zeros, scales, K, bits, g)
    dS = oracle.bwd_ds(d["X"], d["dY"], qw, zeros, bits, g)
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
                ref += (int(codes[i, j]) - int(zeros[i, gi])) * dw
            assert abs(dS[i, gi] - float(ref)) <= 1e-12 * max(1.0, abs(float(ref)))


@pytest.mark.parametrize("bits", [3, 4])
def test_unit_scale_zero_offset_is_integer_matmul(bits):
    """s=1, z=0 and integer activations: Y = X Q^T and dX = dY Q exactly, via int64 matmul."""
    rng = np.random.default_rng(2)
    T, N, K = 17, 24, 96
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    qw = oracle.pack(codes, bits)
    zeros = np.zeros((N, 1), np.uint8)
    scales = np.ones((N, 1), np.float32)
    Xi = rng.integers(-4, 5, size=(T, K))
    dYi = rng.integers(-4, 5, size=(T, N))
    Xb = synth.f32_to_bf16_bits(Xi.astype(np.float32))
    dYb = synth.f32_to_bf16_bits(dYi.astype(np.float32))
    Y = oracle.fwd(Xb, qw, zeros, scales, bits)
    assert np.array_equal(Y, (Xi @ codes.astype(np.int64).T).astype(np.float64))
    dX = oracle.bwd_dx(dYb, qw, zeros, scales, K, bits)
    assert np.array_equal(dX, (dYi @ codes.astype(np.int64)).astype(np.float64))
    dS = oracle.bwd_ds(Xb, dYb, qw, zeros, bits)
    dW = dYi.T @ Xi
    assert np.array_equal(dS[:, 0], (dW * codes.astype(np.int64)).sum(axis=1).astype(np.float64))


def test_matches_dense_float64_matmul():
    """Against numpy's matmul on the explicitly dequantized weight (a library routine as the step)."""
    bits, g = 3, 64
    d, codes, zeros, scales, qw = _case(4, 40, 256, 33, bits, g, sigma_dy=1e-2)
    What = np.repeat(scales.astype(np.float64), g, axis=1) * \
        (codes.astype(np.float64) - np.repeat(zeros.astype(np.float64), g, axis=1))
    X, dY = _f(d["X"]), _f(d["dY"])
    np.testing.assert_allclose(oracle.fwd(d["X"], qw, zeros, scales, bits, g), X @ What.T, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(oracle.bwd_dx(d["dY"], qw, zeros, scales, 256, bits, g), dY @ What, rtol=1e-11, atol=1e-14)
    dW = dY.T @ X
    Wbar = codes.astype(np.float64) - np.repeat(zeros.astype(np.float64), g, axis=1)
    ref = (dW * Wbar).reshape(40, 256 // g, g).sum(axis=2)
    np.testing.assert_allclose(oracle.bwd_ds(d["X"], d["dY"], qw, zeros, bits, g), ref, rtol=1e-10, atol=1e-12)


def test_group_equal_K_is_per_channel():
    d, codes, zeros, scales, qw = _case(5, 16, 128, 9, 4, 0)
    for fn, args in ((oracle.fwd, (d["X"], qw, zeros, scales, 4)),
                     (oracle.bwd_dx, (d["dY"], qw, zeros, scales, 128, 4)),
                     (oracle.bwd_ds, (d["X"], d["dY"], qw, zeros, 4))):
        assert np.array_equal(fn(*args, 0), fn(*args, 128))


@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32)])
def test_scale_gradient_is_finite_difference_of_linear_loss(bits, g):
    """L(s) = <dY, Y(s)> is linear in s, so L(s + e) - L(s) equals dS for a unit step e."""
    d, codes, zeros, scales, qw = _case(6, 12, 64, 7, bits, g)
    dY = _f(d["dY"])
    dS = oracle.bwd_ds(d["X"], d["dY"], qw, zeros, bits, g)
    base = float((dY * oracle.fwd(d["X"], qw, zeros, scales, bits, g)).sum())
    G = scales.shape[1]
    for i in (0, 5, 11):
        for gi in range(G):
            s2 = scales.copy()
            s2[i, gi] += np.float32(1.0)
            step = float(s2[i, gi]) - float(scales[i, gi])      # exactly representable difference
            L = float((dY * oracle.fwd(d["X"], qw, zeros, s2, bits, g)).sum())
            assert abs((L - base) / step - dS[i, gi]) <= 1e-9 * max(1.0, abs(dS[i, gi]))


def test_per_channel_identity_and_adjoint():
    d, codes, zeros, scales, qw = _case(8, 20, 96, 11, 4, 0)
    X, dY = _f(d["X"]), _f(d["dY"])
    Y = oracle.fwd(d["X"], qw, zeros, scales, 4)
    dX = oracle.bwd_dx(d["dY"], qw, zeros, scales, 96, 4)
    dS = oracle.bwd_ds(d["X"], d["dY"], qw, zeros, 4)
    # dS[i] * s[i] = sum_t dY[t,i] Y[t,i]
    np.testing.assert_allclose(dS[:, 0] * scales[:, 0].astype(np.float64), (dY * Y).sum(axis=0), rtol=1e-10, atol=1e-12)
    # <dY, fwd(X)> = <dX, X>
    assert abs((dY * Y).sum() - (dX * X).sum()) <= 1e-10 * abs((dY * Y).sum())


def test_group_with_codes_equal_to_zero_point_is_inert():
    rng = np.random.default_rng(3)
    N, K, g, T = 6, 128, 32, 5
    codes = rng.integers(0, 8, size=(N, K), dtype=np.uint8)
    zeros = rng.integers(0, 8, size=(N, K // g), dtype=np.uint8)
    codes[:, 32:64] = zeros[:, 1:2]
    scales = rng.random((N, K // g), dtype=np.float32) + 0.5
    qw = oracle.pack(codes, 3)
    Xb = synth.f32_to_bf16_bits(rng.standard_normal((T, K)).astype(np.float32))
    dYb = synth.f32_to_bf16_bits(rng.standard_normal((T, N)).astype(np.float32))
    dS = oracle.bwd_ds(Xb, dYb, qw, zeros, 3, g)
    assert np.all(dS[:, 1] == 0.0)
    Y0 = oracle.fwd(Xb, qw, zeros, scales, 3, g)
    s2 = scales.copy()
    s2[:, 1] *= 7.0
    assert np.array_equal(Y0, oracle.fwd(Xb, qw, zeros, s2, 3, g))
    dX = oracle.bwd_dx(dYb, qw, zeros, scales, K, 3, g)
    assert np.all(dX[:, 32:64] == 0.0)


def test_row_and_token_selection_matches_full_result():
    d, codes, zeros, scales, qw = _case(10, 24, 128, 13, 3, 64)
    Y = oracle.fwd(d["X"], qw, zeros, scales, 3, 64)
    dX = oracle.bwd_dx(d["dY"], qw, zeros, scales, 128, 3, 64)
    dS = oracle.bwd_ds(d["X"], d["dY"], qw, zeros, 3, 64)
    tok = [12, 0, 7]
    rows = [23, 1, 8, 8]
    assert np.array_equal(oracle.fwd(d["X"], qw, zeros, scales, 3, 64, tokens=tok), Y[tok])
    assert np.array_equal(oracle.bwd_dx(d["dY"], qw, zeros, scales, 128, 3, 64, tokens=tok), dX[tok])
    assert np.array_equal(oracle.bwd_ds(d["X"], d["dY"], qw, zeros, 3, 64, rows=rows), dS[rows])


def test_bf16_input_conversion_is_round_to_nearest_even():
    a = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38, 1e-40], np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 ties up to 1+2^-6
    b = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(a))
    assert b[0] == 1.0 and b[1] == 1.0 and b[2] == np.float32(1.015625) and b[3] == -2.5
    import torch
    t = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(b, t)


# ---------------------------------------------------------------------------------------------
# Per-channel dS from the stored output: dS[i] = (sum_t dY[t,i] Y[t,i]) / s[i]  (Eq. 2 with G = 1)

@pytest.mark.parametrize("bits", [3, 4])
def test_ds_from_saved_output_equals_ds_when_the_output_is_exact(bits):
    """Power-of-two scales and small integer activations make Y exact in bf16; the two
    routes to dS (through dY^T X, and through the stored Y) must then agree to rounding."""
    rng = np.random.default_rng(5 + bits)
    T, N, K = 23, 12, 64
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    zeros = rng.integers(0, 1 << bits, size=(N, 1), dtype=np.uint8)
    scales = (2.0 ** rng.integers(-3, 2, size=(N, 1))).astype(np.float32)
    qw = oracle.pack(codes, bits)
    # at most two non-zero activations per token keeps |Y| <= 2*15*2 = 60 steps of 1/8: exact in bf16
    Xi = np.zeros((T, K))
    for t in range(T):
        Xi[t, rng.choice(K, 2, replace=False)] = rng.integers(-1, 2, size=2)
    dYi = rng.integers(-3, 4, size=(T, N)).astype(np.float64)
    Xb = synth.f32_to_bf16_bits(Xi.astype(np.float32))
    dYb = synth.f32_to_bf16_bits(dYi.astype(np.float32))
    Y = oracle.fwd(Xb, qw, zeros, scales, bits, 0)
    Yb = synth.f32_to_bf16_bits(Y.astype(np.float32))
    assert np.array_equal(_f(Yb), Y)                      # the premise: nothing was rounded
    a = oracle.bwd_ds(Xb, dYb, qw, zeros, bits, 0)
    b = oracle.bwd_ds_from_y(dYb, Yb, scales)
    assert np.allclose(a, b, rtol=1e-13, atol=1e-13)


def test_ds_from_saved_output_literal_loop_and_rounded_output():
    T, N, K = 40, 9, 128
    d, codes, zeros, scales, qw = _case(11, N, K, T, 4, 0, sigma_dy=1e-2)
    Y = oracle.fwd(d["X"], qw, zeros, scales, 4, 0)
    Yb = synth.f32_to_bf16_bits(Y.astype(np.float32))
    got = oracle.bwd_ds_from_y(d["dY"], Yb, scales)
    dY = _f(d["dY"])
    Yr = _f(Yb)
    for i in range(N):
        ref = sum(Fraction(float(dY[t, i])) * Fraction(float(Yr[t, i])) for t in range(T)) / Fraction(float(scales[i, 0]))
        assert abs(got[i, 0] - float(ref)) <= 1e-12 * max(1.0, abs(float(ref)))
    # against the route through dY^T X: only the bf16 rounding of Y separates them
    full = oracle.bwd_ds(d["X"], d["dY"], qw, zeros, 4, 0)
    err = np.linalg.norm(got - full) / np.linalg.norm(full)
    assert err < 5e-3


# ---------------------------------------------------------------------------------------------
# Zero-point gradient (App. K): dZ[i,g] = -s[i,g] sum_{j in g} (dY^T X)[i,j]

@pytest.mark.parametrize("bits,g", [(4, 0), (3, 32), (4, 64)])
def test_dz_is_the_derivative_of_the_loss_in_a_real_valued_zero_point(bits, g):
    """L(z) = <dY, X W_hat(z)^T> is linear in z, so a finite difference with any step is exact
    up to rounding; W_hat(z) is formed here in numpy fp64 with z made real-valued."""
    T, N, K = 11, 6, 128
    d, codes, zeros, scales, qw = _case(21 + bits + g, N, K, T, bits, g)
    gg = K if g == 0 else g
    G = K // gg
    X, dY = _f(d["X"]), _f(d["dY"])
    s64 = scales.astype(np.float64)

    def loss(z):
        What = np.repeat(s64, gg, axis=1) * (codes.astype(np.float64) - np.repeat(z, gg, axis=1))
        return float(np.sum(dY * (X @ What.T)))

    z0 = zeros.astype(np.float64)
    dZ = oracle.bwd_dz(d["X"], d["dY"], scales, g)
    base = loss(z0)
    for i in range(N):
        for gi in range(G):
            z1 = z0.copy()
            z1[i, gi] += 0.5
            fd = (loss(z1) - base) / 0.5
            assert abs(dZ[i, gi] - fd) <= 1e-9 * max(1.0, abs(fd), abs(base))


def test_dz_through_group_sums_of_the_activations():
    """sum_{j in g} (dY^T X)[i,j] = sum_t dY[t,i] * (sum_{j in g} X[t,j]): the same number by a
    route that never forms dY^T X."""
    T, N, K, g = 19, 8, 192, 64
    d, codes, zeros, scales, qw = _case(31, N, K, T, 3, g)
    X, dY = _f(d["X"]), _f(d["dY"])
    Xg = X.reshape(T, K // g, g).sum(axis=2)                 # [T, G]
    ref = -scales.astype(np.float64) * (dY.T @ Xg)           # [N, G]
    got = oracle.bwd_dz(d["X"], d["dY"], scales, g)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)
    rows = np.array([5, 0, 3], np.int32)
    assert np.allclose(oracle.bwd_dz(d["X"], d["dY"], scales, g, rows=rows), ref[rows], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# Multi-task forward (Sec. 3.3): shared Q and z, task-specific scales

def test_multitask_forward_rows_are_single_task_forwards():
    """Row m equals the plain forward under the scales of task_ids[m]; and since per-channel
    scales factor out of the contraction, Y_task / s_task is the same for every task."""
    T, N, K = 7, 10, 64
    d, codes, zeros, scales, qw = _case(41, N, K, T, 4, 0)
    table = np.stack([scales[:, 0], 2.0 * scales[:, 0], 0.5 * scales[:, 0] + 1e-3]).astype(np.float32)
    ids = np.array([2, 0, 1, 1, 0, 2, 2])
    Y = oracle.fwd_multitask(d["X"], qw, zeros, table, ids, 4)
    X = _f(d["X"])
    u = X @ (codes.astype(np.float64) - zeros.astype(np.float64)).T       # [T, N], scale-free
    for m in range(T):
        assert np.allclose(Y[m], table[ids[m]].astype(np.float64) * u[m], rtol=1e-12, atol=1e-12)
    same = oracle.fwd_multitask(d["X"], qw, zeros, table, np.zeros(T, int), 4)
    assert np.array_equal(same, oracle.fwd(d["X"], qw, zeros, scales, 4, 0))


def test_multitask_forward_with_grouped_scales():
    """Grouped task tables [n_tasks, N, G]: row m is the explicit fp64 product with the weight
    s_task[i, g(j)] * (Q[i, j] - z[i, g(j)]) of its own task."""
    T, N, K, g = 5, 6, 128, 32
    d, codes, zeros, scales, qw = _case(43, N, K, T, 3, g)
    rng = np.random.default_rng(5)
    table = (scales[None] * rng.uniform(0.5, 2.0, size=(3, N, K // g))).astype(np.float32)
    ids = np.array([1, 2, 0, 1, 1])
    Y = oracle.fwd_multitask(d["X"], qw, zeros, table, ids, 3, g)
    X = _f(d["X"])
    centred = codes.astype(np.float64) - np.repeat(zeros.astype(np.float64), g, axis=1)
    for m in range(T):
        W_hat = np.repeat(table[ids[m]].astype(np.float64), g, axis=1) * centred
        assert np.allclose(Y[m], W_hat @ X[m], rtol=1e-12, atol=1e-12)
