"""Inputs and statistics for the joint-independence checks of the shared noise calls.

One Philox call serves eight elements of one rounding slot (16-bit halves of its four words), and the
three slots of an element come from three calls whose counters differ in two bits.  The marginal of
every 16-bit value is tested elsewhere; here the rounding DECISIONS of values that share a word, a
call or an element are tested for independence on inputs whose probability of rounding up is exactly
1/4 in every slot (Eq. 2 with (x - floor) / Delta = 1/4).  Plain numpy, no rounding rule of its own:
the decisions are read off the implementations' outputs.
"""

from __future__ import annotations

import struct

import numpy as np

# FP32 pattern with low half 0x4000: a quarter of the way from one BF16 value to the next
QUARTER_F32_BITS = 0x3F804000          # 1 + 2^-9
QUARTER_DOWN, QUARTER_UP = 0x3F80, 0x3F81


def _f32(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", bits))[0]


# A step of Algorithm 1 whose three results all sit a quarter of the way between two BF16 values:
#   g = 0, m = 2^-50, v = 1, x = 1, beta1 = beta2 = 0.5 (1 + 2^-9)  ->  m' = beta1 2^-50, v' = beta2
#   weight_decay = 1, lr = 1/4 - 2^-10  ->  alpha lambda x = lr exactly; the direction term
#   (about 2^-52) is far below half a spacing of it and is absorbed by the fused multiply-add, so
#   x' = 1 - lr = 0.75 + 2^-10 = 0x3F404000.
QUARTER_STEP_HP = dict(lr=0.25 - 2.0 ** -10, beta1=_f32(0x3F004000), beta2=_f32(0x3F004000), eps=1e-8, weight_decay=1.0)
QUARTER_STEP_STATE_BITS = dict(p=0x3F80, g=0x0000, m=0x2680, v=0x3F80)      # 1, 0, 2^-50, 1 as BF16
QUARTER_STEP_DOWN = dict(p=0x3F40, m=0x2600, v=0x3F00)                       # truncations of x', m', v'


def up_decisions(out_bits: np.ndarray, down_pattern: int) -> np.ndarray:
    """1 where the value moved to the neighbour away from zero, 0 where it was truncated."""
    d = out_bits.astype(np.int64) - down_pattern
    assert set(np.unique(d).tolist()) <= {0, 1}, "output is not one of the two neighbours"
    return d.astype(np.int64)


def chi2_independent_quarters(a: np.ndarray, b: np.ndarray) -> float:
    """Chi-square statistic (3 degrees of freedom) of the 2x2 table of two 0/1 decision arrays against
    the cell probabilities of independent events of probability 1/4 each."""
    n = a.size
    assert b.size == n
    table = np.array([np.count_nonzero((a == i) & (b == j)) for i in (0, 1) for j in (0, 1)], dtype=np.float64)
    expect = n * np.array([9 / 16, 3 / 16, 3 / 16, 1 / 16])
    return float(((table - expect) ** 2 / expect).sum())


CHI2_3DOF_LIMIT = 16.27      # P(chi2_3 > 16.27) = 0.001; inputs are seeded, so a run either passes or fails for good


def pair_tables(up: np.ndarray):
    """Decision pairs inside one slot: (element 2j, element 2j+1) share a word; (element 8k+7, element
    8k+8) sit in consecutive calls; (element i, element i+4) sit in different words of one call."""
    n = up.size - up.size % 8
    u = up[:n]
    same_word = (u[0::2], u[1::2])
    across_calls = (u[7:-1:8], u[8::8])
    g = u.reshape(-1, 8)
    other_word = (g[:, :4].reshape(-1), g[:, 4:].reshape(-1))
    return {"same word": same_word, "consecutive calls": across_calls, "words of one call": other_word}
