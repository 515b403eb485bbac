"""Pins for the oracle's own binary16 conversions (independent of numpy's)."""
import numpy as np

import oracle


def test_f16_roundtrip_exhaustive():
    for bits in range(0x10000):
        e, f = (bits >> 10) & 0x1F, bits & 0x3FF
        v = oracle.f16_to_f32(bits)
        if e == 31 and f:
            assert np.isnan(v)
            continue
        assert oracle.f32_to_f16(v) == bits, hex(bits)


def test_f16_to_f32_matches_format_definition():
    # spot values fixed by the format: 1.0, -2.0, 65504, smallest normal, smallest subnormal
    assert oracle.f16_to_f32(0x3C00) == 1.0
    assert oracle.f16_to_f32(0xC000) == -2.0
    assert oracle.f16_to_f32(0x7BFF) == 65504.0
    assert oracle.f16_to_f32(0x0400) == 2.0 ** -14
    assert oracle.f16_to_f32(0x0001) == 2.0 ** -24
    assert oracle.f16_to_f32(0x3555) == np.float32(np.float16(1.0 / 3.0))


def test_f32_to_f16_rounding_against_numpy_and_ties():
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(5000) * 1e-6).astype(np.float32),   # subnormal range
        (rng.standard_normal(5000) * 3e4).astype(np.float32),    # near overflow
        np.array([65504.0, 65519.9, 65520.0, 1e9, -1e9, 2.0 ** -25, 2.0 ** -25 * 1.0000001,
                  2.0 ** -24 * 1.5, 0.0, -0.0], np.float32),
    ])
    with np.errstate(over="ignore"):
        wants = vals.astype(np.float16).view(np.uint16)
    for v, want in zip(vals, wants):
        want = int(want)
        assert oracle.f32_to_f16(float(v)) == want, float(v)
    # ties go to the even neighbour: 1 + 2^-11 is half way between 1.0 and 1 + 2^-10
    assert oracle.f32_to_f16(1.0 + 2.0 ** -11) == 0x3C00
    assert oracle.f32_to_f16(1.0 + 3 * 2.0 ** -11) == 0x3C02
