"""Pins for the oracle's LoRA bypass (Section 5.5, Table 3): y += LoRA_A (LoRA_B x)."""
import os
from fractions import Fraction

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table3_lora.txt")


def test_bypass_equals_the_other_association_in_exact_rationals():
    # (LoRA_A LoRA_B) x, formed as an explicit [N, K] matrix in Python integers, against LoRA_A (LoRA_B x);
    # M, N, K and r all differ, so a transposed operand cannot pass
    rng = np.random.default_rng(51)
    M, N, K, r = 3, 5, 12, 2
    x = rng.integers(-9, 10, (M, K)).astype(np.float32)
    A = rng.integers(-9, 10, (N, r)).astype(np.float32)
    Bm = rng.integers(-9, 10, (r, K)).astype(np.float32)
    y0 = rng.integers(-50, 51, (M, N)).astype(np.float64)
    got = oracle.lora_bypass(y0, x, A, Bm)
    AB = [[sum(int(A[n, j]) * int(Bm[j, k]) for j in range(r)) for k in range(K)] for n in range(N)]
    for m in range(M):
        for n in range(N):
            want = Fraction(int(y0[m, n])) + sum(Fraction(AB[n][k]) * int(x[m, k]) for k in range(K))
            assert Fraction(got[m, n]) == want


def test_rank_one_closed_form():
    # r = 1: y[m, n] += a[n] * (b . x[m])
    rng = np.random.default_rng(52)
    M, N, K = 2, 7, 40
    x = rng.standard_normal((M, K)).astype(np.float16).astype(np.float32)
    a = rng.standard_normal((N, 1)).astype(np.float16).astype(np.float32)
    b = rng.standard_normal((1, K)).astype(np.float16).astype(np.float32)
    got = oracle.lora_bypass(np.zeros((M, N)), x, a, b)
    for m in range(M):
        dot = sum(Fraction(float(b[0, k])) * Fraction(float(x[m, k])) for k in range(K))
        for n in range(N):
            want = float(Fraction(float(a[n, 0])) * dot)
            assert abs(got[m, n] - want) <= 1e-14 * max(1.0, abs(want))


def test_zero_lora_leaves_y_alone_and_input_is_not_modified():
    y0 = np.arange(12, dtype=np.float64).reshape(3, 4)
    keep = y0.copy()
    x = np.ones((3, 8), np.float32)
    got = oracle.lora_bypass(y0, x, np.zeros((4, 2), np.float32), np.ones((2, 8), np.float32))
    assert (got == keep).all() and (y0 == keep).all()


def test_bypass_adds_to_the_quantised_linear():
    # the whole operation of the path: W4A16 linear + bypass = dense product with (W_hat + A B)
    from paper_2506_10443_b200 import inputs
    M, N, K, r, group = 2, 32, 128, 4, 64
    W = inputs.weights(53, N, K)
    x = inputs.activations(54, M, K).astype(np.float32)
    rng = np.random.default_rng(55)
    A = (rng.standard_normal((N, r)) * 0.05).astype(np.float16).astype(np.float32)
    Bm = (rng.standard_normal((r, K)) * 0.05).astype(np.float16).astype(np.float32)
    q, s, z = oracle.quantize_w4(W, group)
    got = oracle.lora_bypass(oracle.linear_wa16(x, q, s, z, group), x, A, Bm)
    W_hat = oracle.dequant(q, s, z, group)
    want = x.astype(np.float64) @ (W_hat + A.astype(np.float64) @ Bm.astype(np.float64)).T
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()


def test_table3_counts():
    vals = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    h, r = int(vals["h"]), int(vals["r"])
    assert r * h * h + h ** 3 == vals["computation_ab_x"]
    assert 2 * r * h * h == vals["computation_a_bx"]
    assert 2 * (r * h * h + h * h + h ** 3) == vals["memory_ab_x"]
    assert 4 * r * h * h + h * h + r * h == vals["memory_a_bx"]
    ratio = 100.0 * vals["memory_a_bx"] / vals["memory_ab_x"]
    assert abs(ratio - vals["memory_ratio_percent"]) < 1e-3 and round(ratio, 1) == 0.5   # "about 0.5 %"
