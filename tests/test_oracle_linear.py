"""Pins for the oracle's weight-only linear (W4A16 / W8A16)."""
import numpy as np

import oracle
from paper_2506_10443_b200 import inputs


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16)


def brute_force_linear(x, w_hat32):
    """Independent formulation: long-double triple loop over weights dequantised in fp32."""
    M, K = x.shape
    N = w_hat32.shape[0]
    y = np.zeros((M, N), np.longdouble)
    for m in range(M):
        for n in range(N):
            acc = np.longdouble(0)
            for k in range(K):
                acc += np.longdouble(x[m, k]) * np.longdouble(w_hat32[n, k])
            y[m, n] = acc
    return y


def test_tiny_brute_force_w4():
    N, K, M, group = 4, 128, 3, 64     # N != K != M so that a transposed operand cannot pass
    W = inputs.weights(21, N, K)
    x = inputs.activations(22, M, K).astype(np.float32)
    q, s, z = oracle.quantize_w4(W, group)
    # second formulation: expand scale/zero to [N, K] with numpy, dequantise in fp32 products
    S = np.repeat(f16(s).astype(np.float64), group, axis=1)
    Z = np.repeat(f16(z).astype(np.float64), group, axis=1)
    w_hat = S * (q.astype(np.float64) - Z)
    want = brute_force_linear(x, w_hat)
    got = oracle.linear_wa16(x, q, s, z, group)
    assert got.shape == (M, N)
    assert np.abs(got - want.astype(np.float64)).max() <= 1e-12 * np.abs(want).max()


def test_subset_sum_special_case():
    # s = 1, z = 0, q in {0, 1}: y[m, n] is the sum of x[m, k] over the k where q[n, k] == 1
    rng = np.random.default_rng(2)
    N, K, M, group = 5, 192, 2, 64
    q = rng.integers(0, 2, (N, K)).astype(np.uint8)
    s = np.full((N, K // group), 0x3C00, np.uint16)
    z = np.zeros((N, K // group), np.uint16)
    x = inputs.activations(23, M, K).astype(np.float32)
    got = oracle.linear_wa16(x, q, s, z, group)
    for m in range(M):
        for n in range(N):
            assert abs(got[m, n] - x[m, q[n] == 1].astype(np.float64).sum()) < 1e-12


def test_constant_code_closed_form():
    # all codes equal c: y[m, n] = sum_g s[n,g] (c - z[n,g]) * sum_{k in g} x[m, k]
    rng = np.random.default_rng(3)
    N, K, M, group = 3, 256, 2, 128
    G = K // group
    q = np.full((N, K), 11, np.uint8)
    s = rng.uniform(0.001, 0.01, (N, G)).astype(np.float16)
    z = rng.uniform(0, 15, (N, G)).astype(np.float16)
    x = inputs.activations(24, M, K).astype(np.float32)
    got = oracle.linear_wa16(x, q, s.view(np.uint16), z.view(np.uint16), group)
    xs = x.astype(np.float64).reshape(M, G, group).sum(axis=2)
    want = np.einsum("ng,mg->mn", s.astype(np.float64) * (11.0 - z.astype(np.float64)), xs)
    assert np.abs(got - want).max() < 1e-12


def test_group_index_is_along_k_not_n():
    # scale differs per group: zero all but group 1 of row 2 and check only that block contributes
    N, K, M, group = 4, 192, 1, 64
    q = np.full((N, K), 3, np.uint8)
    s = np.zeros((N, 3), np.float16)
    s[2, 1] = 0.5
    z = np.zeros((N, 3), np.float16)
    x = np.arange(K, dtype=np.float32).reshape(1, K) / 8
    got = oracle.linear_wa16(x, q, s.view(np.uint16), z.view(np.uint16), group)
    assert (got[0, [0, 1, 3]] == 0).all()
    assert got[0, 2] == 0.5 * 3 * x[0, 64:128].sum()


def test_w8_per_channel_matches_dense_float_within_quantisation_noise():
    N, K, M = 16, 512, 2
    W = inputs.weights(25, N, K)
    x = inputs.activations(26, M, K).astype(np.float32)
    q, s, z = oracle.quantize_w8(W)
    got = oracle.linear_wa16(x, q, s, z, K)
    dense = x.astype(np.float64) @ W.astype(np.float64).T
    # int8 per channel: error per output ~ N(0, (step/sqrt(12) * |x|_2)^2) plus the fp16 rounding of
    # the zero point (<= 2^-4 codes) times |sum x|; 5 sigma bounds the 32 outputs
    step = f16(s).astype(np.float64).max()
    x2 = np.linalg.norm(x, axis=1).max()
    bound = 5 * step / np.sqrt(12) * x2 + step * 2.0 ** -4 * np.abs(x.sum(axis=1)).max()
    assert np.abs(got - dense).max() < bound
    assert np.abs(got - dense).max() > 0.02 * bound   # and it is not the unquantised product
    w_hat = oracle.dequant(q, s, z, K)
    assert np.abs(got - x.astype(np.float64) @ w_hat.T).max() < 1e-12
