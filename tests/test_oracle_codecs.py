"""Pins of the oracle's number formats and power-of-two helpers.

The oracle decodes and encodes bit patterns by arithmetic.  It is pinned here
against an independent library (PyTorch's CPU casts), against the closed-form
constants of the formats, and against the defining properties of
round-to-nearest-even.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle as orc
import scalify_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

FORMATS = [orc.E4M3, orc.E5M2, orc.F16, orc.BF16]
NBITS = {orc.E4M3: 8, orc.E5M2: 8, orc.F16: 16, orc.BF16: 16}
NP = {orc.E4M3: np.uint8, orc.E5M2: np.uint8, orc.F16: np.uint16, orc.BF16: np.uint16}


def all_patterns(fmt):
    return np.arange(1 << NBITS[fmt], dtype=np.uint32).astype(NP[fmt])


@pytest.mark.parametrize("fmt", FORMATS)
def test_decode_matches_library_for_every_pattern(fmt):
    bits = all_patterns(fmt)
    mine = orc.decode(bits, fmt)
    ref = si.from_bits(bits, fmt)
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])
    assert np.array_equal(np.signbit(mine[ok]), np.signbit(ref[ok]))


@pytest.mark.parametrize("fmt", FORMATS)
def test_encode_inverts_decode_for_every_pattern(fmt):
    bits = all_patterns(fmt)
    vals = orc.decode(bits, fmt)
    back = orc.encode(vals, fmt)
    finite = np.isfinite(vals)
    assert np.array_equal(back[finite], bits[finite])
    # NaN stays NaN
    assert np.all(np.isnan(orc.decode(back[np.isnan(vals)], fmt)))
    inf = np.isinf(vals)
    if fmt in (orc.F16, orc.BF16):
        assert np.array_equal(back[inf], bits[inf])
    elif inf.any():  # E5M2: infinities saturate to the largest finite value
        assert np.array_equal(np.abs(orc.decode(back[inf], fmt)), np.full(inf.sum(), 57344.0))


@pytest.mark.parametrize("fmt", FORMATS)
def test_midpoints_round_to_even_and_neighbours_round_to_nearest(fmt):
    bits = all_patterns(fmt)
    half = 1 << (NBITS[fmt] - 1)
    pos = bits[:half]
    v = orc.decode(pos, fmt)
    keep = np.isfinite(v)
    pos, v = pos[keep], v[keep]
    lo, hi = v[:-1], v[1:]
    assert np.all(hi > lo)  # bit order is value order for positive finite patterns
    mid = (lo + hi) / 2  # exact in fp64
    enc_mid = orc.encode(mid, fmt)
    even = np.where(pos[:-1] % 2 == 0, pos[:-1], pos[1:])
    assert np.array_equal(enc_mid, even)
    # a hair on either side of the midpoint goes to the nearer neighbour; the
    # offsets are far below fp32 resolution, so an encoder that first rounds
    # to fp32 would fail this for BF16/F16
    eps = (hi - lo) * 2.0 ** -30
    assert np.array_equal(orc.encode(mid + eps, fmt), pos[1:])
    assert np.array_equal(orc.encode(mid - eps, fmt), pos[:-1])
    # negatives mirror
    sign = NP[fmt](half)
    assert np.array_equal(orc.encode(-mid, fmt), even | sign)


@pytest.mark.parametrize("fmt", FORMATS)
def test_encode_matches_library_cast_on_random_fp32(fmt):
    rng = np.random.default_rng(11)
    # magnitudes spanning subnormal to near-max of each format, fp32 inputs so
    # that the library cast rounds once
    top = {orc.E4M3: 8.5, orc.E5M2: 15.5, orc.F16: 15.9, orc.BF16: 100.0}[fmt]
    bot = {orc.E4M3: -12.0, orc.E5M2: -19.0, orc.F16: -27.0, orc.BF16: -140.0}[fmt]
    x = (rng.standard_normal(200000) * np.exp2(rng.uniform(bot, top, 200000))).astype(np.float32)
    lim = {orc.E4M3: 448.0, orc.E5M2: 57344.0, orc.F16: 65504.0, orc.BF16: 3.3e38}[fmt]
    x = x[np.abs(x) <= lim]
    ref = si.to_bits(x, fmt)
    mine = orc.encode(x.astype(np.float64), fmt)
    assert np.array_equal(mine, ref)


def test_fp8_constants_golden():
    names = {"E4M3": orc.E4M3, "E5M2": orc.E5M2}
    for line in open(os.path.join(GOLDEN, "fp8_constants.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f, _, hx, val = line.split()
        fmt, bits, v = names[f], int(hx, 16), float(val)
        got = orc.decode_scalar(bits, fmt)
        if math.isnan(v):
            assert math.isnan(got)
        else:
            assert got == v
            if math.isfinite(v):
                assert orc.encode_scalar(v, fmt) == bits


def test_fp8_overflow_saturates_and_wide_formats_overflow_to_inf():
    assert orc.encode_scalar(1e9, orc.E4M3) == 0x7E
    assert orc.encode_scalar(-1e9, orc.E4M3) == 0xFE
    assert orc.encode_scalar(float("inf"), orc.E4M3) == 0x7E
    assert orc.encode_scalar(465.0, orc.E4M3) == 0x7E  # would round to 480, not representable
    assert orc.encode_scalar(464.0, orc.E4M3) == 0x7E  # tie between 448 and 480 -> even mantissa 110
    assert orc.encode_scalar(1e9, orc.E5M2) == 0x7B
    assert orc.encode_scalar(float("inf"), orc.E5M2) == 0x7B
    assert orc.encode_scalar(61440.0, orc.E5M2) == 0x7B  # tie 57344/65536 -> would be inf; saturates
    assert orc.encode_scalar(65520.0, orc.F16) == 0x7C00  # IEEE: rounds to 2^16 -> inf
    assert orc.encode_scalar(65519.0, orc.F16) == 0x7BFF
    assert orc.encode_scalar(float("inf"), orc.BF16) == 0x7F80
    assert orc.encode_scalar(3.4e38, orc.BF16) == 0x7F80
    assert math.isnan(orc.decode_scalar(orc.encode_scalar(float("nan"), orc.E4M3), orc.E4M3))
    assert math.isnan(orc.decode_scalar(orc.encode_scalar(float("nan"), orc.F16), orc.F16))
    assert orc.encode_scalar(-0.0, orc.BF16) == 0x8000


def test_f32_codec_is_ieee_binary32():
    x = np.array([0.1, -1e-45, 3.4028235e38, 1e39, 2.0 ** -149 * 0.5, 2.0 ** -149 * 0.5000001])
    bits = orc.encode(x, orc.F32)
    ref = x.astype(np.float32).view(np.uint32)
    assert np.array_equal(bits, ref)
    assert np.array_equal(orc.decode(bits, orc.F32), ref.view(np.float32).astype(np.float64))


def test_p2f_is_floor_to_power_of_two_for_every_exponent():
    for e in range(-149, 128):
        p = math.ldexp(1.0, e)
        assert orc.p2f(p) == p
        assert orc.p2f(p * 1.9999999) == p
        assert orc.p2f(p * 1.5) == p
        if e > -149:
            assert orc.p2f(math.nextafter(p, 0.0)) == p / 2
    assert orc.p2f(0.02) == 2.0 ** -6
    assert orc.p2f(3e-4) == 2.0 ** -12
    assert orc.p2f(1e-8) == 2.0 ** -27


def test_kf_golden_table_and_closed_form():
    for line in open(os.path.join(GOLDEN, "kf_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        K, f = line.split()
        assert orc.kf(int(K)) == float(f), K
    # kf(K) = largest power of two <= sqrt(K); check with integer arithmetic
    for K in list(range(1, 5000)) + [2 ** 20 - 1, 2 ** 20, 2 ** 21, 2 ** 31 + 5]:
        f = int(orc.kf(K))
        assert f & (f - 1) == 0
        assert f * f <= K < (2 * f) * (2 * f)
