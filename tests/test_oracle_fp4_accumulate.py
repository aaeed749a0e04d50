"""Pins for two more uses of Eq. 2 in the oracle: the 4-bit grid E2M1 and a BF16 accumulator.

E2M1: the eight magnitudes are typed in from the format's definition and cross-checked against the
exponent/mantissa formula; neighbours are found by value; the rounding threshold gives exactly
P(up) = (|x| - floor)/Delta and an exact mean.  Accumulation: the FP32 sum is checked against correctly
rounded exact rational arithmetic, the rounding by enumerating all 65536 noise values (exact mean),
and Section 2.1's stagnation example is replayed over many steps."""

import bisect
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from exact import bf16_neighbours, bits_f32, f32_bits, frac_of_bf16_bits, frac_of_f32_bits, round_to_f32_bits

E2M1 = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def test_e2m1_table_follows_the_format_definition():
    for code, val in enumerate(E2M1):
        e, man = code >> 1, code & 1
        want = Fraction(man, 2) if e == 0 else (1 + Fraction(man, 2)) * Fraction(2) ** (e - 1)   # bias 1
        assert val == want
    assert E2M1 == sorted(E2M1)


_XS = [1.0, 1.25, -1.25, 0.1, 0.25, 0.4999999, 0.75, 1.7, 2.5, -2.9, 3.5, 5.0, 5.999999, 4.0, 1e-3, 3e-9, 1e-30,
       bits_f32(0x3F800001), bits_f32(0x3FFFFFFF), bits_f32(0x3F000001), bits_f32(0x00000001), bits_f32(0x00800000)]


@pytest.mark.parametrize("x", _XS)
def test_eq2_on_the_e2m1_grid(x):
    fb = f32_bits(x)
    xq = frac_of_f32_bits(fb)
    sign = 8 if xq < 0 else 0
    i = bisect.bisect_right(E2M1, abs(xq)) - 1
    lo = i
    if E2M1[i] == abs(xq):
        for r in (0, 1, 0x7FFFFFFF, 0xFFFFFFFF):
            assert oracle.sr_fp4_bits(fb, r) == sign | lo
        return
    hi = lo + 1
    delta = E2M1[hi] - E2M1[lo]
    T = (abs(xq) - E2M1[lo]) / delta * (1 << 32)
    exact = T.denominator == 1
    T = T.numerator // T.denominator
    rng = np.random.default_rng(fb & 0xFFFF)
    for r in [0, T - 1, T, T + 1, 0xFFFFFFFF] + [int(v) for v in rng.integers(0, 1 << 32, 200)]:
        if 0 <= r <= 0xFFFFFFFF:
            assert oracle.sr_fp4_bits(fb, r) == sign | (hi if r < T else lo)
    mean = E2M1[lo] + delta * Fraction(T, 1 << 32)
    assert (mean == abs(xq)) if exact else (0 < abs(xq) - mean < delta * Fraction(1, 1 << 32))
    if x in (1.25, 0.1, 2.5, 5.0, 1e-3):
        assert exact


def test_e2m1_special_values():
    for r in (0, 0xFFFFFFFF):
        assert oracle.sr_fp4_bits(0x00000000, r) == 0 and oracle.sr_fp4_bits(0x80000000, r) == 8
        assert oracle.sr_fp4_bits(f32_bits(6.0), r) == 7 and oracle.sr_fp4_bits(f32_bits(-6.0), r) == 15
        assert oracle.sr_fp4_bits(f32_bits(6.5), r) == 7 and oracle.sr_fp4_bits(f32_bits(-1e30), r) == 15
        assert oracle.sr_fp4_bits(0x7F800000, r) == 7 and oracle.sr_fp4_bits(0xFF800000, r) == 15     # infinity saturates
        assert oracle.sr_fp4_bits(0x7FC00000, r) == 7 and oracle.sr_fp4_bits(0xFFC00001, r) == 15     # NaN: largest magnitude
    # between 4 and 6 the upper level is reachable, beyond 6 nothing above it exists
    assert oracle.sr_fp4_bits(f32_bits(5.0), 0) == 7 and oracle.sr_fp4_bits(f32_bits(5.0), 0xFFFFFFFF) == 6


def test_e2m1_array_packing_and_noise():
    seed, step, tid = (5 << 32) | 17, 9, 2
    rng = np.random.default_rng(8)
    src = (rng.normal(0, 1, 1001) * 10.0 ** rng.uniform(-3, 1, 1001)).astype(np.float32)
    out = oracle.sr_downcast_fp4(src, seed, step, tid, elem_offset=21)
    assert out.shape == (501,) and out[500] >> 4 == 0          # odd length: upper half of the last byte is 0
    for i in list(range(0, 1001, 13)) + [999, 1000]:
        code = (out[i >> 1] >> (4 * (i & 1))) & 0xF
        assert code == oracle.sr_fp4_bits(f32_bits(float(src[i])), oracle.noise32(seed, step, tid, 21 + i))
    again = oracle.sr_downcast_fp4(np.ascontiguousarray(src[100:200]), seed, step, tid, elem_offset=121)
    assert np.array_equal(again, out[50:100])


def test_e2m1_is_unbiased_in_the_mean_over_many_draws():
    x = np.full(1 << 16, 2.3, dtype=np.float32)
    out = oracle.sr_downcast_fp4(x, seed=3)
    codes = np.stack([out & 0xF, out >> 4], axis=1).reshape(-1)
    assert set(np.unique(codes)) == {4, 5}                       # 2 and 3
    p_up = (codes == 5).mean()
    assert abs(p_up - 0.3) < 6 * np.sqrt(0.3 * 0.7 / codes.size)   # (2.3 - 2) / 1


# ---------------------------------------------------------------------------------------------
# accumulation
# ---------------------------------------------------------------------------------------------

def test_slot_layout_of_the_noise():
    seed, step, tid = (11 << 32) | 5, 1234, 6
    for idx in (0, 1, 6, 7, 8, 1001, (1 << 35) + 3):
        assert [oracle.noise_slot(seed, step, tid, idx, s) for s in range(3)] == list(oracle.noise(seed, step, tid, idx))
        number = 4 * (idx >> 3) + 3
        w = oracle.philox4x32_10([number & 0xFFFFFFFF, number >> 32, tid, seed >> 32], [seed & 0xFFFFFFFF, step])
        word = w[(idx & 7) >> 1]
        assert oracle.noise_slot(seed, step, tid, idx, 3) == ((word >> 16) if idx & 1 else (word & 0xFFFF))


_ACC_CASES = [(0x3F80, 2.0 ** -9, 1.0), (0x3F80, 0.001, 1.0), (0xBF80, 0.001, 0.125), (0x0000, 3.1e-5, 1.0),
              (0x4049, -1e-3, 0.5), (0x3A83, 7.7e-4, 1.0 / 3.0), (0x7F7F, 1e36, 1.0), (0x0001, 1e-41, 1.0),
              (0x3F80, -1.0, 1.0), (0xC2C8, 100.0, 1.0)]


@pytest.mark.parametrize("acc,g,scale", _ACC_CASES)
def test_accumulation_sum_and_rounding_are_exact(acc, g, scale):
    gq, sq = frac_of_f32_bits(f32_bits(g)), frac_of_f32_bits(f32_bits(scale))
    t_bits = round_to_f32_bits(gq * sq)
    s_bits = round_to_f32_bits(frac_of_bf16_bits(acc) + frac_of_f32_bits(t_bits))
    if s_bits & 0x7FFFFFFF == 0:                                  # exact cancellation: +0 under round-to-nearest
        s_bits = 0
    lo, up = bf16_neighbours(s_bits)
    low16 = s_bits & 0xFFFF
    outs = [oracle.accumulate_element(acc, g, scale, r, True) for r in range(0, 65536, 1 if low16 else 4096)]
    assert set(outs) <= {lo, up}
    if low16:
        assert sum(o == up for o in outs) == low16                # P(up) = low16 / 65536
        if up & 0x7FFF <= 0x7F7F:                                 # both neighbours finite: the mean is the FP32 sum
            mean = (frac_of_bf16_bits(lo) * (65536 - low16) + frac_of_bf16_bits(up) * low16) / 65536
            assert mean == frac_of_f32_bits(s_bits)
    # nearest rounding returns the closer neighbour
    near = oracle.accumulate_element(acc, g, scale, 0, False)
    assert near == oracle.rne_bf16_bits(s_bits) and near in (lo, up)


def test_stagnation_example_over_many_accumulations(golden_dir):
    """Section 2.1: a term far below the spacing never moves a nearest-rounded accumulator, while under
    Q_SR the accumulator follows the exact sum on average."""
    gold = dict(line.split(" = ") for line in open(os.path.join(golden_dir, "paper_examples.txt")).read().splitlines()
                if line and not line.startswith("#"))
    assert gold["stagnation_nearest_returns_x"] == "1" and gold["stagnation_sr_mean_is_x_plus_u"] == "1"
    n, steps, u = 4096, 256, 2.0 ** -9                           # spacing at 1.0 is 2^-7: u is a quarter of it
    g = np.full(n, u, dtype=np.float32)
    near = np.full(n, 0x3F80, dtype=np.uint16)
    sr = near.copy()
    for t in range(1, steps + 1):
        oracle.sr_accumulate(near, g, 1.0, seed=99, step=t, stochastic=False)
        oracle.sr_accumulate(sr, g, 1.0, seed=99, step=t, stochastic=True)
    assert np.all(near == 0x3F80)                                 # stagnation
    vals = (sr.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    exact = 1.0 + steps * u                                       # 1.5
    # each step's error has variance Delta^2 q (1 - q) <= Delta^2 / 4 with Delta <= 2^-7
    sigma = np.sqrt(steps * (2.0 ** -7) ** 2 / 4)
    assert abs(vals.mean() - exact) < 6 * sigma / np.sqrt(n)
    assert vals.std() > 0.2 * sigma


def test_accumulate_array_driver_and_shard_invariance():
    rng = np.random.default_rng(12)
    n = 3000
    acc0 = (rng.normal(0, 1e-2, n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    g32 = rng.normal(0, 1e-3, n).astype(np.float32)
    g16 = (g32.view(np.uint32) >> 16).astype(np.uint16)
    seed, step, tid = 1234, 7, 3
    for g in (g32, g16):
        full = oracle.sr_accumulate(acc0.copy(), g, 0.25, seed, step, tid, elem_offset=40)
        for i in range(0, n, 41):
            gi = float(g[i]) if g.dtype == np.float32 else bits_f32(int(g[i]) << 16)
            r = oracle.noise_slot(seed, step, tid, 40 + i, 3)
            assert full[i] == oracle.accumulate_element(int(acc0[i]), gi, 0.25, r, True)
        part = oracle.sr_accumulate(acc0[1000:2000].copy(), np.ascontiguousarray(g[1000:2000]), 0.25, seed, step, tid,
                                    elem_offset=1040)
        assert np.array_equal(part, full[1000:2000])
        other = oracle.sr_accumulate(acc0.copy(), g, 0.25, seed, step + 1, tid, elem_offset=40)
        assert not np.array_equal(other, full)
