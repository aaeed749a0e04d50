"""Pins for the oracle's FP8 stochastic rounding (Eq. 2 on the E4M3 / E5M2 grids): the level tables
are built from the formats' definitions and checked against a library's decode; neighbours are found
by value; the rounding threshold gives exactly P(up) = (x - floor)/Delta and an exact mean."""

import bisect
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from exact import bits_f32, f32_bits, frac_of_f32_bits


def _levels(e5m2: bool):
    """Non-negative finite levels by code, from the format definition."""
    M, bias = (2, 15) if e5m2 else (3, 7)
    out = {}
    for code in range(0x80):
        e, man = code >> M, code & ((1 << M) - 1)
        if e5m2 and e == 31:
            continue                                   # infinity and NaNs
        if not e5m2 and code == 0x7F:
            continue                                   # the single NaN of E4M3
        if e == 0:
            out[code] = Fraction(man, 1 << M) * Fraction(2) ** (1 - bias)
        else:
            out[code] = (1 + Fraction(man, 1 << M)) * Fraction(2) ** (e - bias)
    return out


@pytest.mark.parametrize("e5m2", [False, True])
def test_level_table_matches_library_decode(e5m2):
    dtype = torch.float8_e5m2 if e5m2 else torch.float8_e4m3fn
    lv = _levels(e5m2)
    codes = torch.arange(256, dtype=torch.uint8)
    dec = codes.view(dtype).to(torch.float32).numpy()
    for code, val in lv.items():
        assert Fraction(float(dec[code])) == val and Fraction(float(dec[code | 0x80])) == -val
    assert max(lv.values()) == (57344 if e5m2 else 448)
    assert sorted(lv, key=lv.get) == sorted(lv)       # codes are ordered like values


def _neighbours(x: Fraction, lv):
    codes = sorted(lv)
    vals = [lv[c] for c in codes]
    i = bisect.bisect_right(vals, abs(x)) - 1
    lo = codes[i]
    hi = lo if vals[i] == abs(x) else codes[i + 1]
    return lo, hi


_XS = [1.0, 1.1, -1.1, 0.3333333433, 447.9, 300.0, 0.0019531, 0.001, 1e-3 + 1e-9, -2.5e-3, 0.0175, 3.0517578125e-05,
       1.7e-5, 6e-8, 57343.0, 40000.0, 1.5258789e-05, bits_f32(0x3F800001), bits_f32(0x3FFFFFFF), bits_f32(0x3C000001)]


@pytest.mark.parametrize("e5m2", [False, True])
@pytest.mark.parametrize("x", _XS)
def test_eq2_on_the_fp8_grid(x, e5m2):
    lv = _levels(e5m2)
    top = max(lv.values())
    fb = f32_bits(x)
    xq = frac_of_f32_bits(fb)
    if abs(xq) >= top:
        assert oracle.sr_fp8_bits(fb, 0, e5m2) & 0x7F == (0x7B if e5m2 else 0x7E)
        return
    lo, hi = _neighbours(xq, lv)
    sign = 0x80 if xq < 0 else 0
    if lo == hi:
        for r in (0, 1, 0x7FFFFFFF, 0xFFFFFFFF):
            assert oracle.sr_fp8_bits(fb, r, e5m2) == sign | lo
        return
    delta = lv[hi] - lv[lo]
    T = (abs(xq) - lv[lo]) / delta * (1 << 32)           # P(up) * 2^32
    exact = T.denominator == 1                           # at most 32 fractional bits: exactly unbiased
    T = T.numerator // T.denominator                     # otherwise the probability is rounded down by < 2^-32
    # only the two neighbours occur; the move happens exactly for the T smallest noise values
    rng = np.random.default_rng(fb & 0xFFFF)
    for r in [0, T - 1, T, T + 1, 0xFFFFFFFF] + [int(v) for v in rng.integers(0, 1 << 32, 200)]:
        if 0 <= r <= 0xFFFFFFFF:
            want = hi if r < T else lo
            assert oracle.sr_fp8_bits(fb, r, e5m2) == sign | want
    # hence P(up) = T / 2^32 = (|x| - floor) / Delta and the mean is x
    mean = lv[lo] + delta * Fraction(T, 1 << 32)
    assert (mean == abs(xq)) if exact else (0 < abs(xq) - mean < delta * Fraction(1, 1 << 32))
    if x in (1.1, 300.0, 0.0175, 40000.0):
        assert exact


@pytest.mark.parametrize("e5m2", [False, True])
def test_fp8_special_values(e5m2):
    top = 0x7B if e5m2 else 0x7E
    for r in (0, 0xFFFFFFFF):
        assert oracle.sr_fp8_bits(0x00000000, r, e5m2) == 0x00 and oracle.sr_fp8_bits(0x80000000, r, e5m2) == 0x80
        assert oracle.sr_fp8_bits(0x7FC00000, r, e5m2) == 0x7F and oracle.sr_fp8_bits(0xFF800001, r, e5m2) == 0x7F
        assert oracle.sr_fp8_bits(0x7F800000, r, e5m2) == (0x7C if e5m2 else 0x7E)
        assert oracle.sr_fp8_bits(0xFF800000, r, e5m2) == (0xFC if e5m2 else 0xFE)
        assert oracle.sr_fp8_bits(f32_bits(1e30), r, e5m2) == top and oracle.sr_fp8_bits(f32_bits(-1e30), r, e5m2) == 0x80 | top
    # far below the smallest level: up only for the very smallest noise values
    tiny = f32_bits(1e-30)
    assert oracle.sr_fp8_bits(tiny, 0xFFFFFFFF, e5m2) == 0 and oracle.sr_fp8_bits(tiny, 1 << 20, e5m2) == 0


@pytest.mark.parametrize("e5m2", [False, True])
def test_library_nearest_cast_lands_on_one_of_the_two_levels(e5m2):
    dtype = torch.float8_e5m2 if e5m2 else torch.float8_e4m3fn
    rng = np.random.default_rng(5)
    x = (rng.normal(0, 1, 3000) * 10.0 ** rng.uniform(-4, 2, 3000)).astype(np.float32)
    x = x[np.abs(x) < (57344 if e5m2 else 448)]
    near = torch.from_numpy(x).to(dtype).view(torch.uint8).numpy()
    for xi, ni in zip(x.tolist(), near.tolist()):
        fb = f32_bits(xi)
        assert ni in (oracle.sr_fp8_bits(fb, 0, e5m2), oracle.sr_fp8_bits(fb, 0xFFFFFFFF, e5m2))


def test_noise32_layout_and_array_driver():
    seed, step, tid = (7 << 32) | 9, 3, 11
    for idx in (0, 1, 2, 3, 4, 1023, (1 << 34) + 6):
        number = idx >> 2
        w = oracle.philox4x32_10([number & 0xFFFFFFFF, number >> 32, tid, seed >> 32], [seed & 0xFFFFFFFF, step])
        assert oracle.noise32(seed, step, tid, idx) == w[idx & 3]
    rng = np.random.default_rng(6)
    src = (rng.normal(0, 1, 1000) * 10.0 ** rng.uniform(-6, 3, 1000)).astype(np.float32)
    for e5m2 in (False, True):
        out = oracle.sr_downcast_fp8(src, e5m2, seed, step, tid, elem_offset=13)
        for i in range(0, 1000, 37):
            assert out[i] == oracle.sr_fp8_bits(f32_bits(float(src[i])), oracle.noise32(seed, step, tid, 13 + i), e5m2)
        again = oracle.sr_downcast_fp8(np.ascontiguousarray(src[100:200]), e5m2, seed, step, tid, elem_offset=113)
        assert np.array_equal(again, out[100:200])
