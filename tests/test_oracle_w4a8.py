"""Pins for the oracle's W4A8 path: activation quantiser, integer group partials, rescale."""
from fractions import Fraction

import numpy as np

import oracle
from paper_2506_10443_b200 import inputs


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16)


def test_act_quant_hand_rows():
    K, group = 128, 64
    x = np.zeros((3, K), np.float32)
    # row 0: amax = 127 -> inv = 1, a_scale = 1, codes are the rounded values (half to even)
    x[0, :6] = (127.0, -3.0, 2.5, 3.5, -0.5, 64.0)
    x[0, 64] = -127.0
    # row 1: amax = 2 -> inv = 63.5; 1.0 -> 63.5 -> 64 (even), 0.5 -> 31.75 -> 32, -2 -> -127
    x[1, :3] = (1.0, 0.5, -2.0)
    # row 2: all zero
    a_q, a_scale, A_g = oracle.act_quant(x, group)
    assert list(a_q[0, :6]) == [127, -3, 2, 4, 0, 64] and a_q[0, 64] == -127
    assert a_scale[0] == 1.0
    assert list(A_g[0]) == [127 - 3 + 2 + 4 + 0 + 64, -127]
    assert list(a_q[1, :3]) == [64, 32, -127] and a_scale[1] == np.float32(2.0) / np.float32(127.0)
    assert (a_q[2] == 0).all() and a_scale[2] == 0.0 and (A_g[2] == 0).all()


def test_act_quant_range_and_error_bound():
    x = inputs.activations(31, 5, 1536, outliers=True).astype(np.float32)
    a_q, a_scale, A_g = oracle.act_quant(x, 64)
    assert a_q.min() >= -127 and a_q.max() <= 127
    for m in range(5):
        amax = np.abs(x[m]).max()
        assert abs(int(a_q[m, np.abs(x[m]).argmax()])) == 127
        assert a_scale[m] == np.float32(amax) / np.float32(127)
        assert np.abs(a_q[m] * np.float64(a_scale[m]) - x[m]).max() <= 0.5 * a_scale[m] * (1 + 1e-5)
    assert (A_g == a_q.astype(np.int64).reshape(5, -1, 64).sum(axis=2)).all()


def test_group_partials_brute_force_integers():
    rng = np.random.default_rng(7)
    M, N, K, group = 3, 5, 128, 64
    a_q = rng.integers(-127, 128, (M, K)).astype(np.int8)
    q = rng.integers(0, 16, (N, K)).astype(np.uint8)
    P = oracle.group_partials(a_q, q, group)
    assert P.shape == (M, N, K // group) and P.dtype == np.int32
    for m in range(M):
        for n in range(N):
            for g in range(K // group):
                want = sum(int(a_q[m, k]) * int(q[n, k]) for k in range(g * group, (g + 1) * group))
                assert int(P[m, n, g]) == want
    # extreme values stay inside int32: 127 * 15 * 128
    P2 = oracle.group_partials(np.full((1, 128), -127, np.int8), np.full((1, 128), 15, np.uint8), 128)
    assert int(P2[0, 0, 0]) == -127 * 15 * 128


def test_group_identity_in_exact_rationals():
    # sum_k a * s * (q - z) == s * (sum_k a*q - z * sum_k a), per group, in exact arithmetic
    rng = np.random.default_rng(8)
    group = 64
    a = [int(v) for v in rng.integers(-127, 128, group)]
    q = [int(v) for v in rng.integers(0, 16, group)]
    s = Fraction(float(np.float16(0.00731)))
    z = Fraction(float(np.float16(7.43)))
    lhs = sum(Fraction(ai) * s * (Fraction(qi) - z) for ai, qi in zip(a, q))
    rhs = s * (sum(ai * qi for ai, qi in zip(a, q)) - z * sum(a))
    assert lhs == rhs


def test_w4a8_matches_rational_evaluation():
    M, N, K, group = 2, 3, 128, 64
    W = inputs.weights(32, N, K)
    x = inputs.activations(33, M, K, outliers=True).astype(np.float32)
    q, s, z = oracle.quantize_w4(W, group)
    a_q, a_scale, A_g = oracle.act_quant(x, group)
    got = oracle.linear_w4a8(x, q, s, z, group)
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                g = k // group
                acc += Fraction(int(a_q[m, k])) * Fraction(float(f16(s)[n, g])) * (
                    Fraction(int(q[n, k])) - Fraction(float(f16(z)[n, g])))
            want = float(Fraction(float(a_scale[m])) * acc)
            assert abs(got[m, n] - want) <= 1e-13 * max(1.0, abs(want))


def test_w4a8_equals_w4a16_when_activations_are_int8_exact():
    # integer activations with amax = 127: a_scale = 1, a_q = x, so both paths are the same sum
    rng = np.random.default_rng(9)
    M, N, K, group = 3, 6, 256, 64
    x = rng.integers(-127, 128, (M, K)).astype(np.float32)
    x[:, 0] = 127
    W = inputs.weights(34, N, K)
    q, s, z = oracle.quantize_w4(W, group)
    y8 = oracle.linear_w4a8(x, q, s, z, group)
    y16 = oracle.linear_wa16(x, q, s, z, group)
    assert np.abs(y8 - y16).max() <= 1e-12 * np.abs(y16).max()


def test_w4a8_close_to_w4a16_on_gaussian_activations():
    # int8 activations: relative error ~ 1 / (127 * sqrt(12)) * (amax / rms); a wrong a_scale or a
    # dropped zero-point term is off by orders of magnitude more
    M, N, K, group = 4, 64, 1536, 64
    x = inputs.activations(35, M, K).astype(np.float32)
    W = inputs.weights(36, N, K)
    q, s, z = oracle.quantize_w4(W, group)
    y8 = oracle.linear_w4a8(x, q, s, z, group)
    y16 = oracle.linear_wa16(x, q, s, z, group)
    rel = np.linalg.norm(y8 - y16) / np.linalg.norm(y16)
    assert rel < 0.02, rel
