"""Pins for the oracle's quantised-KV attention (Section 4.2: int8 keys, fp8 values; Section 5.4)."""
import math

import numpy as np

import oracle


def e4m3_value(b):
    """The E4M3 format written out: 1 sign, 4 exponent bits (bias 7), 3 fraction bits, no infinities."""
    sign = -1.0 if b & 0x80 else 1.0
    e, f = (b >> 3) & 15, b & 7
    if e == 15 and f == 7:
        return math.nan
    if e == 0:
        return sign * f * 2.0 ** -9
    return sign * (1 + f / 8.0) * 2.0 ** (e - 7)


def test_e4m3_all_bit_patterns_and_round_trip():
    for b in range(256):
        want, got = e4m3_value(b), oracle.e4m3_to_f32(b)
        if math.isnan(want):
            assert math.isnan(got)
            continue
        assert got == want
        assert oracle.f32_to_e4m3(got) == (b if want != 0 or b == 0 else b)   # -0 keeps its sign bit
    assert oracle.e4m3_to_f32(0x7E) == 448.0 and oracle.e4m3_to_f32(0x01) == 2.0 ** -9
    assert oracle.e4m3_to_f32(0x38) == 1.0


def test_e4m3_rounding_ties_and_saturation():
    # between 1.0 (0x38) and 1.125 (0x39): below the midpoint, the tie (even fraction wins), above
    assert oracle.f32_to_e4m3(1.06) == 0x38
    assert oracle.f32_to_e4m3(1.0625) == 0x38
    assert oracle.f32_to_e4m3(1.07) == 0x39
    # between 1.125 (0x39, odd) and 1.25 (0x3A, even): the tie goes up
    assert oracle.f32_to_e4m3(1.1875) == 0x3A
    # subnormals: 2^-10 is the tie between 0 and 2^-9 -> 0; 3 * 2^-10 between 2^-9 (odd) and 2^-8 -> 2^-8
    assert oracle.f32_to_e4m3(2.0 ** -10) == 0x00
    assert oracle.f32_to_e4m3(3 * 2.0 ** -10) == 0x02
    # saturation and sign
    assert oracle.f32_to_e4m3(1e9) == 0x7E and oracle.f32_to_e4m3(-500.0) == 0xFE
    assert oracle.f32_to_e4m3(464.0) == 0x7E and oracle.f32_to_e4m3(float("inf")) == 0x7E
    assert oracle.f32_to_e4m3(-1.0) == 0xB8


def cache(seed, Hk, S, D):
    rng = np.random.default_rng(seed)
    k = rng.standard_normal((Hk, S, D)).astype(np.float32)
    v = rng.standard_normal((Hk, S, D)).astype(np.float32)
    kc, ks, kz = oracle.quantize_keys(k)
    return kc, ks, kz, oracle.quantize_values(v)


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


def test_attention_brute_force_tiny():
    # every step written out with Python floats: dequantised keys, scaled query, softmax, weighted values
    H, Hk, S, D = 4, 2, 5, 8
    kc, ks, kz, vb = cache(91, Hk, S, D)
    q = np.random.default_rng(92).standard_normal((H, D)).astype(np.float16).astype(np.float32)
    got = oracle.attention_decode(q, kc, ks, kz, vb)
    for h in range(H):
        hk = h // (H // Hk)
        scores = []
        for t in range(S):
            s, z = float(f16(ks)[hk, t]), float(f16(kz)[hk, t])
            scores.append(sum(float(q[h, d]) / math.sqrt(D) * (s * (int(kc[hk, t, d]) - z)) for d in range(D)))
        mx = max(scores)
        w = [math.exp(x - mx) for x in scores]
        for d in range(D):
            want = sum(w[t] / sum(w) * e4m3_value(int(vb[hk, t, d])) for t in range(S))
            assert abs(got[h, d] - want) <= 1e-12 * max(1.0, abs(want))


def test_equal_keys_give_the_mean_of_the_values():
    H, Hk, S, D = 2, 1, 7, 16
    kc, ks, kz, vb = cache(93, Hk, S, D)
    kc[:], ks[:], kz[:] = kc[0, 0], ks[0, 0], kz[0, 0]     # every token carries the same key
    q = np.random.default_rng(94).standard_normal((H, D)).astype(np.float32)
    got = oracle.attention_decode(q, kc, ks, kz, vb)
    vals = np.vectorize(e4m3_value)(vb.astype(int))[0]
    assert np.abs(got - vals.mean(axis=0)).max() <= 1e-13


def test_one_key_far_ahead_gives_its_value():
    H, Hk, S, D = 1, 1, 6, 8
    kc, ks, kz, vb = cache(95, Hk, S, D)
    q = np.full((H, D), 30.0, np.float32)
    kc[:] = 0
    kz[:] = np.array([0.0], np.float16).view(np.uint16)
    ks[:] = np.array([1.0], np.float16).view(np.uint16)
    kc[0, 3] = 255        # score of token 3: 30 * 255 * 8 / sqrt(8), all others 0
    got = oracle.attention_decode(q, kc, ks, kz, vb)
    assert (got[0] == np.vectorize(e4m3_value)(vb[0, 3].astype(int))).all()


def test_group_query_mapping_and_zero_point_shift_invariance():
    # query heads 0..2 read kv head 0, heads 3..5 kv head 1; adding a constant to every key of a head
    # shifts all its scores alike and leaves the softmax unchanged (here: the zero point of each key,
    # moved by a multiple that keeps s * z * sum(q) equal over tokens because all scales are equal)
    H, Hk, S, D = 6, 2, 9, 16
    kc, ks, kz, vb = cache(96, Hk, S, D)
    ks[:] = np.array([0.03125], np.float16).view(np.uint16)
    q = np.random.default_rng(97).standard_normal((H, D)).astype(np.float16).astype(np.float32)
    base = oracle.attention_decode(q, kc, ks, kz, vb)
    assert np.abs(base[:3] - oracle.attention_decode(q[:3], kc[:1], ks[:1], kz[:1], vb[:1])).max() == 0.0
    assert np.abs(base[3:] - oracle.attention_decode(q[3:], kc[1:], ks[1:], kz[1:], vb[1:])).max() == 0.0
    kz2 = kz.copy()
    kz2[:] = np.array([64.0], np.float16).view(np.uint16)
    kz[:] = np.array([3.0], np.float16).view(np.uint16)
    a = oracle.attention_decode(q, kc, ks, kz, vb)
    b = oracle.attention_decode(q, kc, ks, kz2, vb)
    assert np.abs(a - b).max() <= 1e-12


def test_key_quantisation_is_eq1_per_key_vector():
    k = np.random.default_rng(98).standard_normal((2, 3, 16)).astype(np.float32)
    kc, ks, kz = oracle.quantize_keys(k)
    assert kc.shape == (2, 3, 16) and ks.shape == (2, 3)
    for hk in range(2):
        for t in range(3):
            assert kc[hk, t].min() == 0 and kc[hk, t].max() == 255          # the end points of Eq. 1
            back = f16(ks)[hk, t] * (kc[hk, t].astype(np.float64) - f16(kz)[hk, t])
            assert np.abs(back - k[hk, t]).max() <= 0.51 * f16(ks)[hk, t] + 2e-3 * np.abs(k[hk, t]).max()
