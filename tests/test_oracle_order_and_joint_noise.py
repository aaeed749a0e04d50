"""Two pins of the oracle that nothing else gives without a GPU.

1. The ORDER of the fixed summation tree (the squared norm's contract): a plain restatement of the rule
   as the library header words it, compared bit for bit on data where the order of the additions
   changes the rounded result -- and shown to be order-sensitive by planting three mistakes in the
   restatement (loops swapped, a running sum instead of the butterfly, groups added in reverse).
2. Joint behaviour of rounding decisions that share a Philox call: elements that share a word, words
   of one call, consecutive calls, and the three slots (x, m, v) of one element are pairwise
   independent at P(up) = 1/4 (chi-square on 2x2 tables over 2^20 indices).
"""

import numpy as np
import pytest

import joint
import oracle


# ---------------------------------------------------------------------------------------------
# summation tree, restated from the header's wording
# ---------------------------------------------------------------------------------------------

def _block_sum(terms: np.ndarray, swap_loops=False, running_sum=False, reverse_groups=False) -> float:
    """One block of at most 8192 doubles: 256 accumulators, accumulator j adding entries r*1024 + 4j + k
    for r = 0..7 and, inside r, k = 0..3, in that order (missing entries skipped); 8 groups of 32
    accumulators, each folded by exchanging with the partner at distance 16, 8, 4, 2, 1; the 8 group
    values added in order 0..7.  All 256 accumulators advance together, one addition each per step."""
    padded = np.zeros(8192, dtype=np.float64)
    present = np.zeros(8192, dtype=bool)
    padded[:terms.size] = terms
    present[:terms.size] = True
    j = np.arange(256)
    acc = np.zeros(256, dtype=np.float64)
    order = [(r, k) for k in range(4) for r in range(8)] if swap_loops else [(r, k) for r in range(8) for k in range(4)]
    for r, k in order:
        e = r * 1024 + 4 * j + k
        acc = np.where(present[e], acc + padded[e], acc)
    groups = acc.reshape(8, 32)
    if running_sum:
        folded = np.array([float(np.cumsum(g)[-1]) for g in groups])      # left-to-right sum: a mistake
    else:
        lanes = groups.copy()
        for s in (16, 8, 4, 2, 1):
            lanes = lanes + lanes[:, np.arange(32) ^ s]
        assert all(len(set(row.tolist())) == 1 for row in lanes)          # every lane ends with the same value
        folded = lanes[:, 0]
    total = 0.0
    first = True
    for w in (range(7, -1, -1) if reverse_groups else range(8)):
        total = float(folded[w]) if first else total + float(folded[w])
        first = False
    return total


def _tree(terms: np.ndarray, **mistake) -> float:
    level = np.asarray(terms, dtype=np.float64)
    if level.size == 0:
        return 0.0
    while True:
        level = np.array([_block_sum(level[s:s + 8192], **mistake) for s in range(0, level.size, 8192)])
        if level.size == 1:
            return float(level[0])


def _spread_f32(n: int, seed: int, octaves: int = 20) -> np.ndarray:
    """FP32 values with magnitudes spread over 2^-octaves .. 2^octaves (their squares over twice that),
    shuffled.  The wide spread makes small terms vanish or survive depending on what was added before
    them; the narrow one makes every single addition round."""
    rng = np.random.default_rng(seed)
    g = (rng.uniform(1.0, 2.0, n) * np.exp2(rng.integers(-octaves, octaves + 1, n)) * rng.choice([-1.0, 1.0], n)).astype(np.float32)
    rng.shuffle(g)
    return g


def _datasets(n: int):
    return [_spread_f32(n, 1000 + n, 20), _spread_f32(n, 2000 + n, 2), _spread_f32(n, 3000 + n, 6)]


_SIZES = [5, 8191, 8193, 3 * 8192 + 77, 8192 * 8192 // 64 + 77]


@pytest.mark.parametrize("n", _SIZES)
def test_summation_order_is_the_headers(n):
    for g in _datasets(n):
        squares = g.astype(np.float64) ** 2                               # exact: 24-bit significands
        want = _tree(squares)
        assert oracle.sqnorm(g).hex() == want.hex()
        assert oracle.tree_sum(squares).hex() == want.hex()
        # BF16 input takes the same route
        gb = (g.view(np.uint32) >> 16).astype(np.uint16)
        sq16 = (gb.astype(np.uint32) << 16).view(np.float32).astype(np.float64) ** 2
        assert oracle.sqnorm(gb).hex() == _tree(sq16).hex()
        # block by block: the final value of a long array hides most single-block differences
        for start in range(0, min(n, 40 * 8192), 8192):
            assert oracle.sqnorm(g[start:start + 8192].copy()).hex() == _block_sum(squares[start:start + 8192]).hex()


def test_list_norm_order_is_the_headers():
    """Block sums per chunk of each tensor (positions counted from the chunk's start), then the tree over them."""
    sizes = [5, 8191, 8193, 3 * 8192 + 77, 1, 20000]
    grads = [_spread_f32(n, 2000 + i) for i, n in enumerate(sizes)]
    partials = [_block_sum(g.astype(np.float64)[s:s + 8192] ** 2) for g in grads for s in range(0, g.size, 8192)]
    assert oracle.sqnorm_list(grads).hex() == _tree(np.array(partials)).hex()


@pytest.mark.parametrize("mistake", ["swap_loops", "running_sum", "reverse_groups"])
def test_the_data_tell_the_orders_apart(mistake):
    """The pin above would be empty if every order gave the same bits on its data.  Each planted
    mistake changes more than a tenth of the block sums that the pin compares, so an oracle with that
    mistake fails the pin many times over."""
    blocks = changed = 0
    for n in _SIZES[1:]:
        for g in _datasets(n):
            sq = g.astype(np.float64) ** 2
            for start in range(0, min(n, 40 * 8192), 8192):
                blocks += 1
                changed += _block_sum(sq[start:start + 8192], **{mistake: True}).hex() != _block_sum(sq[start:start + 8192]).hex()
    assert changed > 0.1 * blocks, (changed, blocks)


# ---------------------------------------------------------------------------------------------
# decisions that share a Philox call
# ---------------------------------------------------------------------------------------------

N_JOINT = 1 << 20


def test_cast_decisions_inside_and_across_calls_are_independent():
    src = np.full(N_JOINT, np.uint32(joint.QUARTER_F32_BITS)).view(np.float32)
    up = joint.up_decisions(oracle.sr_downcast(src, seed=11, step=3, tensor_id=2), joint.QUARTER_DOWN)
    assert abs(up.mean() - 0.25) < 4 * np.sqrt(0.1875 / N_JOINT)
    for name, (a, b) in joint.pair_tables(up).items():
        assert joint.chi2_independent_quarters(a, b) < joint.CHI2_3DOF_LIMIT, name


def test_step_decisions_of_the_three_slots_are_independent():
    st = joint.QUARTER_STEP_STATE_BITS
    p, g, m, v = (np.full(N_JOINT, st[k], dtype=np.uint16) for k in ("p", "g", "m", "v"))
    oracle.adamw_step(p, g, m, v, oracle.hparams(**joint.QUARTER_STEP_HP), seed=(5 << 32) | 9, step=1, tensor_id=4)
    up = {k: joint.up_decisions(a, joint.QUARTER_STEP_DOWN[k]) for k, a in (("p", p), ("m", m), ("v", v))}
    for k, u in up.items():
        assert abs(u.mean() - 0.25) < 4 * np.sqrt(0.1875 / N_JOINT), k
        for name, (a, b) in joint.pair_tables(u).items():
            assert joint.chi2_independent_quarters(a, b) < joint.CHI2_3DOF_LIMIT, (k, name)
    for a, b in (("p", "m"), ("m", "v"), ("p", "v")):
        assert joint.chi2_independent_quarters(up[a], up[b]) < joint.CHI2_3DOF_LIMIT, (a, b)
    # a slot of one element against the next slot of its neighbour in the same word
    assert joint.chi2_independent_quarters(up["p"][0::2], up["m"][1::2]) < joint.CHI2_3DOF_LIMIT


def test_the_statistic_sees_shared_bits():
    """Planted mistake: if both elements of a word used the SAME half, or two slots the same call, the
    table would be far from independent; the statistic must say so."""
    rng = np.random.default_rng(3)
    a = (rng.random(N_JOINT) < 0.25).astype(np.int64)
    assert joint.chi2_independent_quarters(a, a) > 1e5
    b = np.where(rng.random(N_JOINT) < 0.05, a, (rng.random(N_JOINT) < 0.25).astype(np.int64))   # 5 % shared
    assert joint.chi2_independent_quarters(a, b) > joint.CHI2_3DOF_LIMIT
