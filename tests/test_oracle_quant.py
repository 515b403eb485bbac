"""Pins for the oracle's weight quantiser and dequantiser (Eq. 1, Section 4.2)."""
import os

import numpy as np
import pytest

import oracle
from paper_2506_10443_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


def test_worked_group_from_golden_file():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "eq1_worked_group.txt"))
            if l.strip() and not l.startswith("#")]
    w = np.array([[float(r[0]) for r in rows]], np.float32)
    want = np.array([int(r[2]) for r in rows], np.uint8)
    assert w.shape[1] == 16
    q, s, z = oracle.quantize_w4(w, 16)
    assert f16(s)[0, 0] == 0.25 and f16(z)[0, 0] == 6.0
    assert (q[0] == want).all()
    # and the codes are what the file's middle column rounds to (half to even)
    t = np.array([float(r[1]) for r in rows])
    assert (np.rint(t) == want).all()


def test_scale_and_zero_saturate_at_fp16_max_golden_file():
    for line in open(os.path.join(GOLDEN, "eq1_saturation.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        w, sb, zb, codes = [f.split() for f in line.split("|")]
        q, s, z = oracle.quantize_w4(np.array([[float(v) for v in w]], np.float32), 4)
        assert s[0, 0] == int(sb[0], 16) and z[0, 0] == int(zb[0], 16), line
        assert q[0].tolist() == [int(c) for c in codes], line


@pytest.mark.parametrize("group", [64, 128])
def test_eq1_endpoints_and_monotone(group):
    W = inputs.weights(11, 24, 4 * group)
    q, s, z = oracle.quantize_w4(W, group)
    assert q.min() == 0 and q.max() == 15
    Wg = W.reshape(24, 4, group)
    qg = q.reshape(24, 4, group)
    for n in range(24):
        for g in range(4):
            w, c = Wg[n, g], qg[n, g]
            assert c[w.argmin()] == 0 and c[w.argmax()] == 15   # w_min -> clip_min, w_max -> clip_max
            order = np.argsort(w, kind="stable")
            assert (np.diff(c[order].astype(int)) >= 0).all()   # monotone in w
            # scale is fp16((max-min)/15) and zero is fp16(-min/scale)
            sc = np.float32(np.float16((w.max() - w.min()) / np.float32(15)))
            assert f16(s)[n, g] == sc
            assert f16(z)[n, g] == np.float16(-w.min() / sc)
            # each code is the nearest level: |w - w_hat| <= s/2 (+ fp32 rounding slack)
            w_hat = sc * (c.astype(np.float64) - f16(z)[n, g])
            zero_err = abs(float(np.float16(-w.min() / sc)) - float(-w.min() / sc)) * sc
            assert np.abs(w - w_hat).max() <= sc / 2 * (1 + 1e-5) + zero_err + 1e-9


@pytest.mark.parametrize("group,levels", [(64, 15), (128, 15)])
def test_lossless_roundtrip_int4(group, levels):
    rng = np.random.default_rng(5)
    N, G = 9, 3
    W = np.empty((N, G * group), np.float32)
    for n in range(N):
        for g in range(G):
            s = float(np.float16(2.0 ** rng.integers(-9, -3) * (1 + rng.integers(0, 8) / 8)))
            zero = float(rng.integers(0, 16))            # integer zero => -min/s exact in fp16
            i = rng.integers(0, levels + 1, group)
            i[:2] = (0, levels)                          # the group must span all codes
            rng.shuffle(i)
            W[n, g * group:(g + 1) * group] = (i - zero) * s
            assert ((i - zero) * s == W[n, g * group:(g + 1) * group]).all()
    q, sb, zb = oracle.quantize_w4(W, group)
    w_hat = oracle.dequant(q, sb, zb, group)
    assert (w_hat == W.astype(np.float64)).all()


def test_lossless_roundtrip_int8_per_channel():
    rng = np.random.default_rng(6)
    N, K = 7, 512
    W = np.empty((N, K), np.float32)
    for n in range(N):
        s = float(np.float16(2.0 ** rng.integers(-9, -3) * (1 + rng.integers(0, 8) / 8)))
        zero = float(rng.integers(0, 256))
        i = rng.integers(0, 256, K)
        i[:2] = (0, 255)
        rng.shuffle(i)
        W[n] = (i - zero) * s
    q, sb, zb = oracle.quantize_w8(W)
    assert q.min() == 0 and q.max() == 255
    assert (oracle.dequant(q, sb, zb, K) == W.astype(np.float64)).all()


def test_degenerate_groups():
    W = np.zeros((2, 128), np.float32)
    W[0, :64] = 0.375          # constant group
    W[0, 64:] = 0.0            # all-zero group
    W[1, :64] = np.linspace(0, 1e-9, 64, dtype=np.float32)  # range below fp16 resolution
    W[1, 64:] = -2.5
    q, s, z = oracle.quantize_w4(W, 64)
    assert (q == 0).all()
    assert (f16(s) == 1.0).all()
    assert f16(z)[0, 0] == -0.375 and f16(z)[0, 1] == 0.0 and f16(z)[1, 1] == 2.5
    w_hat = oracle.dequant(q, s, z, 64)
    assert (w_hat[0] == W[0]).all() and (w_hat[1, 64:] == -2.5).all()


def test_quantisation_noise_matches_uniform_quantiser_theory():
    # N(0, sigma) in groups of 64: range ~ 2 * 2.36 sigma, step = range / 15, rms error = step / sqrt(12)
    W = inputs.weights(3, 256, 1536)
    q, s, z = oracle.quantize_w4(W, 64)
    rel = np.linalg.norm(oracle.dequant(q, s, z, 64) - W) / np.linalg.norm(W)
    assert 0.07 < rel < 0.11, rel


def test_table1_shapes_used_by_the_workloads():
    kv = dict(l.split() for l in open(os.path.join(GOLDEN, "table1_qwen2_7b.txt"))
              if l.strip() and not l.startswith("#"))
    assert inputs.QWEN2_7B["hidden"] == int(kv["hidden_size"])
    assert inputs.QWEN2_7B["inter"] == int(kv["intermediate_size"])
    assert inputs.QWEN2_7B["layers"] == int(kv["layers"])
    assert inputs.LM_HEAD["K"] == int(kv["hidden_size"])
    # bf16 embedding: vocab * hidden * 2 bytes = 1.087e9 ("1.09"); one row = 7168 B ("7 KB")
    emb = int(kv["vocabulary_size"]) * int(kv["hidden_size"]) * 2
    assert round(emb / 1e9, 2) == float(kv["embedding_size_printed_1e9"])
    assert int(kv["hidden_size"]) * 2 == int(kv["embedding_row_bytes_bf16"])
