"""Pins for the oracle's per-channel W8A8 path (Section 4.2: int8 weights, int8 activations)."""
from fractions import Fraction

import numpy as np

import oracle
from paper_2506_10443_b200 import inputs


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16)


def test_w8a8_brute_force_in_exact_rationals():
    # every output written out as a_scale * sum_k a_q * s * (q - z) with Python integers and Fractions
    M, N, K = 3, 4, 96
    W = inputs.weights(41, N, K)
    x = inputs.activations(42, M, K, outliers=True).astype(np.float32)
    q, s, z = oracle.quantize_w8(W)
    a_q, a_scale, _ = oracle.act_quant(x, K)
    got = oracle.linear_w8a8(x, q, s, z)
    assert got.shape == (M, N) and got.dtype == np.float64
    for m in range(M):
        for n in range(N):
            sn, zn = Fraction(float(f16(s)[n, 0])), Fraction(float(f16(z)[n, 0]))
            acc = sum(Fraction(int(a_q[m, k])) * sn * (Fraction(int(q[n, k])) - zn) for k in range(K))
            want = float(Fraction(float(a_scale[m])) * acc)
            assert abs(got[m, n] - want) <= 1e-13 * max(1.0, abs(want))


def test_w8a8_equals_w8a16_when_activations_are_int8_exact():
    # integer activations with amax = 127: a_scale = 1 and a_q = x, so both paths are the same sum
    rng = np.random.default_rng(43)
    M, N, K = 3, 7, 320
    x = rng.integers(-127, 128, (M, K)).astype(np.float32)
    x[:, 5] = -127
    W = inputs.weights(44, N, K)
    q, s, z = oracle.quantize_w8(W)
    y8 = oracle.linear_w8a8(x, q, s, z)
    y16 = oracle.linear_wa16(x, q, s, z, K)
    assert np.abs(y8 - y16).max() <= 1e-12 * np.abs(y16).max()


def test_w8a8_constant_code_closed_form():
    # all codes of a row equal c: y = a_scale * s * (c - z) * sum_k a_q, whatever the activations
    rng = np.random.default_rng(45)
    M, N, K = 2, 3, 160
    x = rng.standard_normal((M, K)).astype(np.float32)
    q = np.empty((N, K), np.uint8)
    q[0], q[1], q[2] = 0, 255, 131
    s = np.array([[0.0123], [0.5], [2.0 ** -9]], np.float16).view(np.uint16)
    z = np.array([[17.25], [128.0], [0.0]], np.float16).view(np.uint16)
    a_q, a_scale, A = oracle.act_quant(x, K)
    got = oracle.linear_w8a8(x, q, s, z)
    for m in range(M):
        for n, c in enumerate((0, 255, 131)):
            want = float(a_scale[m]) * float(f16(s)[n, 0]) * (c - float(f16(z)[n, 0])) * int(A[m, 0])
            assert abs(got[m, n] - want) <= 1e-12 * max(1e-3, abs(want))


def test_w8a8_is_the_group_formula_with_one_group_per_row():
    # the W4A8 rescale with group = K and 8-bit codes is the same expression
    M, N, K = 4, 9, 256
    W = inputs.weights(46, N, K)
    x = inputs.activations(47, M, K).astype(np.float32)
    q, s, z = oracle.quantize_w8(W)
    assert np.abs(oracle.linear_w8a8(x, q, s, z) - oracle.linear_w4a8(x, q, s, z, K)).max() == 0.0


def test_w8a8_extreme_codes_do_not_overflow():
    # |sum a_q q| reaches 127 * 255 * K: beyond int32 from K = 66312 on; the sum is kept in 64 bits
    K = 70000
    x = np.full((1, K), -3.0, np.float32)           # a_q = -127 everywhere, a_scale = 3 / 127
    q = np.full((1, K), 255, np.uint8)
    s = np.array([[1.0]], np.float16).view(np.uint16)
    z = np.array([[0.0]], np.float16).view(np.uint16)
    got = oracle.linear_w8a8(x, q, s, z)
    want = float(np.float32(3.0) / np.float32(127.0)) * (-127 * 255 * K)
    assert abs(got[0, 0] - want) <= 1e-12 * abs(want)


def test_w8a8_close_to_dense_float_on_gaussian_data():
    # int8 weights and activations: the result stays within quantisation noise of the fp64 product;
    # a wrong a_scale, a dropped zero-point term or a transposed operand is off by far more
    M, N, K = 4, 48, 1536
    x = inputs.activations(48, M, K).astype(np.float32)
    W = inputs.weights(49, N, K)
    q, s, z = oracle.quantize_w8(W)
    y8 = oracle.linear_w8a8(x, q, s, z)
    dense = x.astype(np.float64) @ W.astype(np.float64).T
    rel = np.linalg.norm(y8 - dense) / np.linalg.norm(dense)
    assert rel < 0.03, rel
