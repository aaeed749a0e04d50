"""Pins for the oracle's random bits and rounding rules: the Philox authors' known-answer vectors,
Eq. 2 (two neighbours, exact probability, exact mean, exact variance) by enumerating all 65536
noise values, Eq. 1 against a library cast, and the worked examples of Section 2."""

import bisect
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from exact import (bits_f32, f32_bits, frac_of_bf16_bits, frac_of_f32_bits, is_inf_bits, is_nan_bits)


# ---------------------------------------------------------------------------------------------
# Philox4x32-10
# ---------------------------------------------------------------------------------------------

def _kat_rows(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat_rows(golden_dir)
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(oracle.philox4x32_10(ctr, key)) == out


def test_philox_is_sensitive_to_every_input_word():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] ^= 1
        assert oracle.philox4x32_10(c, [5, 6]) != base
    for i in range(2):
        k = [5, 6]
        k[i] ^= 1
        assert oracle.philox4x32_10([1, 2, 3, 4], k) != base


def _expected_noise(seed, step, tid, idx):
    """Noise layout written out: one call per (group of 8 elements, rounding slot)."""
    group, e = idx >> 3, idx & 7
    out = []
    for slot in range(3):
        number = 4 * group + slot
        w = oracle.philox4x32_10([number & 0xFFFFFFFF, number >> 32, tid, seed >> 32], [seed & 0xFFFFFFFF, step])
        word = w[e >> 1]
        out.append((word >> 16) if e & 1 else (word & 0xFFFF))
    return tuple(out)


def test_noise_layout_key_counter_and_words():
    """key = (seed low, step); counter = (number low, number high, tensor_id, seed high) with
    number = 4 * (index >> 3) + slot; element e = index & 7 uses word e >> 1, low half if e is even."""
    seed, step, tid = 0x1234_5678_9ABC_DEF0, 77, 9
    for idx in ((5 << 32) | 0xFFFF_FFF3, (5 << 32) | 0xFFFF_FFF8, (1 << 33) - 1, 1 << 33, (1 << 61) + 5, 0, 1, 7, 8):
        assert oracle.noise(seed, step, tid, idx) == _expected_noise(seed, step, tid, idx)


def test_a_group_of_eight_uses_every_bit_once():
    """The eight elements of a group reproduce, slot by slot, all four words of that slot's call."""
    for base in (0, 8, 8 * 10**12):
        got = [oracle.noise(3, 4, 5, base + e) for e in range(8)]
        for slot in range(3):
            number = 4 * (base >> 3) + slot
            w = oracle.philox4x32_10([number & 0xFFFFFFFF, number >> 32, 5, 0], [3, 4])
            words = [got[2 * j][slot] | (got[2 * j + 1][slot] << 16) for j in range(4)]
            assert tuple(words) == w


def test_noise_streams_differ():
    ref = [oracle.noise(1, 1, 0, i) for i in range(64)]
    assert [oracle.noise(2, 1, 0, i) for i in range(64)] != ref            # seed
    assert [oracle.noise(1, 2, 0, i) for i in range(64)] != ref            # iteration
    assert [oracle.noise(1, 1, 1, i) for i in range(64)] != ref            # tensor
    assert [oracle.noise(1 | (1 << 32), 1, 0, i) for i in range(64)] != ref  # high half of the seed
    assert [oracle.noise(1, 1, 0, i + (1 << 33)) for i in range(64)] != ref  # high half of the call number
    assert len(set(ref)) == 64


def test_noise_is_uniform_on_16_bits():
    n = 1 << 16
    vals = np.array([oracle.noise(7, 0, 0, i) for i in range(n)], dtype=np.int64)
    assert vals.min() >= 0 and vals.max() < 65536
    for col in range(3):
        counts = np.bincount(vals[:, col] >> 8, minlength=256)   # 256 bins, expectation 256 each
        chi2 = float(((counts - 256.0) ** 2 / 256.0).sum())
        assert chi2 < 400.0                                      # 255 dof: mean 255, sd ~22.6


# ---------------------------------------------------------------------------------------------
# Eq. 2
# ---------------------------------------------------------------------------------------------

_POS_BF16 = [frac_of_bf16_bits(h) for h in range(0x0000, 0x7F80)]   # all finite non-negative BF16, ascending


def _floor_ceil_by_value(x: Fraction):
    """Largest BF16 <= x and smallest BF16 >= x, found by searching the full list of BF16 values
    (definition of the two quantisation levels around x in Eq. 2).  Returns Fractions."""
    a = abs(x)
    assert a <= _POS_BF16[-1]
    i = bisect.bisect_right(_POS_BF16, a) - 1
    lo_mag = _POS_BF16[i]
    hi_mag = lo_mag if lo_mag == a else _POS_BF16[i + 1]
    if x >= 0:
        return lo_mag, hi_mag
    return -hi_mag, -lo_mag


_GRID = [
    1.0 + 2.0 ** -12, -3.14159274, 1e-40, -1e-40, 2.0 ** -6 - 2.0 ** -30, 2.0 - 2.0 ** -23, 0.3333333433,
    -0.02, 6e-4, 1.1754946e-38, 1.1754942e-38, 3.0e38, -65504.0, 1.00390625 + 2.0 ** -20,
    bits_f32(0x00000001), bits_f32(0x0000FFFF), bits_f32(0x00010001), bits_f32(0x007FFFFF),
    bits_f32(0x3F7FFFFF), bits_f32(0xBF80FFFF), bits_f32(0x7F7EFFFF), bits_f32(0x3F808000), bits_f32(0x3F818000),
]


@pytest.mark.parametrize("x", _GRID)
def test_eq2_by_enumeration(x):
    fb = f32_bits(x)
    xq = frac_of_f32_bits(fb)
    floor_v, ceil_v = _floor_ceil_by_value(xq)
    delta = ceil_v - floor_v
    assert delta > 0
    outs = np.array([oracle.sr_bf16_bits(fb, r) for r in range(65536)], dtype=np.int64)
    vals = {int(h): frac_of_bf16_bits(int(h)) for h in np.unique(outs)}
    # (a) only the two adjacent levels occur
    assert set(vals.values()) <= {floor_v, ceil_v}
    # (d) P(ceil) = (x - floor) / Delta, exactly
    n_ceil = sum(int((outs == h).sum()) for h, val in vals.items() if val == ceil_v)
    assert Fraction(n_ceil, 65536) == (xq - floor_v) / delta
    # (c) the mean over all noise values is x, exactly
    mean = sum(Fraction(int((outs == h).sum()), 65536) * val for h, val in vals.items())
    assert mean == xq
    # quantisation-error lemma: E[r^2] = Delta^2 q (1 - q)
    q = (xq - floor_v) / delta
    var = sum(Fraction(int((outs == h).sum()), 65536) * (val - xq) ** 2 for h, val in vals.items())
    assert var == delta * delta * q * (1 - q)
    # the number of "away from zero" outcomes is the low half of the pattern, and grows with r
    away = outs != (fb >> 16)
    assert int(away.sum()) == (fb & 0xFFFF)
    assert np.all(np.diff(away.astype(np.int8)) >= 0)


def test_eq2_passthrough_of_representable_values():
    rng = np.random.default_rng(0)
    pats = [0x0000, 0x8000, 0x7F80, 0xFF80, 0x0001, 0x8001, 0x007F, 0x0080, 0x3F80, 0xBF80, 0x7F7F, 0xFF7F]
    pats += [int(h) for h in rng.integers(0, 1 << 16, 300)]
    for h in pats:
        fb = h << 16
        if is_nan_bits(fb):
            continue
        for r in (0, 1, 0x7FFF, 0x8000, 0xFFFF):
            assert oracle.sr_bf16_bits(fb, r) == h


def test_nan_stays_nan_and_is_canonical():
    for fb in (0x7FC00000, 0xFFC00000, 0x7F800001, 0xFF800001, 0x7FFFFFFF, 0xFFFFFFFF, 0x7F80FFFF, 0x7FBF0000):
        for r in (0, 1, 0xFFFF):
            assert oracle.sr_bf16_bits(fb, r) == 0x7FC0
        assert oracle.rne_bf16_bits(fb) == 0x7FC0


def test_beyond_largest_bf16_dithers_to_infinity():
    """Above the largest finite BF16 the upper level is infinity: reached for low16 of the 65536
    noise values, like any other carry."""
    fb = 0x7F7F1000
    outs = [oracle.sr_bf16_bits(fb, r) for r in range(65536)]
    assert set(outs) == {0x7F7F, 0x7F80}
    assert outs.count(0x7F80) == 0x1000
    assert oracle.sr_bf16_bits(fb | 0x80000000, 0xFFFF) == 0xFF80


def test_stagnation_example():
    """Section 2.1: u << x.  Nearest rounding of x + u gives x back; the SR mean is x + u."""
    x, u = 1.0, 2.0 ** -12
    fb = f32_bits(x + u)
    assert frac_of_f32_bits(fb) == Fraction(1) + Fraction(1, 4096)          # x + u is exact in FP32
    assert oracle.rne_bf16_bits(fb) == f32_bits(x) >> 16
    mean = sum(frac_of_bf16_bits(oracle.sr_bf16_bits(fb, r)) for r in range(65536)) / 65536
    assert mean == Fraction(1) + Fraction(1, 4096)


def test_random_walk_example():
    """Section 2.2: two consecutive levels, half-step updates twice, then epsilon-steps.
    P(T <= 2) = 3/4 and P(T = n) = 1/4 (1-eps)^(n-3) eps for n >= 3."""
    lo = 0x3F80                                    # 1.0; next BF16 level is 1 + 2^-7
    hi = lo + 1
    delta = frac_of_bf16_bits(hi) - frac_of_bf16_bits(lo)
    half = f32_bits(float(frac_of_bf16_bits(lo) + delta / 2))
    eps = Fraction(1, 16)
    small = f32_bits(float(frac_of_bf16_bits(lo) + delta * eps))
    p_half = Fraction(sum(oracle.sr_bf16_bits(half, r) == hi for r in range(65536)), 65536)
    p_eps = Fraction(sum(oracle.sr_bf16_bits(small, r) == hi for r in range(65536)), 65536)
    assert p_half == Fraction(1, 2) and p_eps == eps
    p_T_le_2 = p_half + (1 - p_half) * p_half
    assert p_T_le_2 == Fraction(3, 4)
    for n in (3, 4, 7):
        p_T_n = (1 - p_half) ** 2 * (1 - p_eps) ** (n - 3) * p_eps
        assert p_T_n == Fraction(1, 4) * (1 - eps) ** (n - 3) * eps


# ---------------------------------------------------------------------------------------------
# Eq. 1
# ---------------------------------------------------------------------------------------------

def test_nearest_rounding_matches_library_cast():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 1 << 32, 200000, dtype=np.uint64).astype(np.uint32)
    ties = (rng.integers(0, 1 << 16, 2000, dtype=np.uint64).astype(np.uint32) << 16) | 0x8000
    bits = np.concatenate([bits, ties, np.array([0x7F7F8000, 0x7F7F7FFF, 0x00008000, 0x00007FFF], dtype=np.uint32)])
    t = torch.from_numpy(bits.view(np.int32)).view(torch.float32)
    lib_cast = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for fb, want in zip(bits.tolist(), lib_cast.tolist()):
        got = oracle.rne_bf16_bits(fb)
        if is_nan_bits(fb):
            assert got == 0x7FC0 and (want & 0x7F80) == 0x7F80 and (want & 0x7F) != 0
        else:
            assert got == want


def test_nearest_rounding_is_nearest():
    """Eq. 1: the result is the BF16 value closest to x (checked by value)."""
    rng = np.random.default_rng(2)
    for fb in rng.integers(0, 0x7F000000, 300).tolist():
        xq = frac_of_f32_bits(fb)
        floor_v, ceil_v = _floor_ceil_by_value(xq)
        got = frac_of_bf16_bits(oracle.rne_bf16_bits(fb))
        assert got in (floor_v, ceil_v)
        assert abs(got - xq) == min(abs(floor_v - xq), abs(ceil_v - xq))
    assert not is_inf_bits(oracle.rne_bf16_bits(0x7F7F7FFF) << 16)
