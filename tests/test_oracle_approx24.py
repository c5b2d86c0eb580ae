"""Pins for the oracle's approx-MVUE 2:4 sampler against what Sec. 4.4 fixes: the two sequential
magnitude-proportional draws, the inclusion-probability equation, unbiasedness, and the scan of
the variance ratio against the optimal estimator (bounded below two, largest where one element
dominates); plus zero rules, validity of every outcome and planted mistakes."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import theory

RNG = np.random.Generator(np.random.PCG64(2203))

BLOCKS = [
    [1, 2, 3, 4], [1, 2, 3, 5.5], [1, 1, 1, 10], [-1, 1, -1, 1], [1, 2, 3, 6], [4, 3, 2, 1],
    [3, -1, 4, -1.5], [10, 1, 1, 1], [1, 10, 1, 1], [0, 1, 2, 3], [0, 1, 1, 1], [1e-3, 1e3, 1.0, 1.0],
    [2, 2, 2, 2], [0.25, -7, 0.5, 1e-2],
]


def random_blocks(n):
    out = []
    for _ in range(n):
        kind = RNG.integers(0, 3)
        if kind == 0:
            a = RNG.standard_normal(4)
        elif kind == 1:
            a = np.exp(2 * RNG.standard_normal(4)) * RNG.choice([-1, 1], 4)
        else:
            a = RNG.standard_t(3, 4) * 1e-3
        out.append(list(a))
    return out


# ------------------------------------------------------------------ theory vs the paper ---
@pytest.mark.parametrize("block", BLOCKS + random_blocks(20))
def test_equation_equals_enumeration_over_ordered_pairs(block):
    # the numbered equation of Sec. 4.4 is the probability of being drawn first or second
    law = theory.approx24_ordered_law(block)
    assert math.isclose(law.sum(), 1.0, rel_tol=1e-12)
    p_enum = law.sum(0) + law.sum(1)
    p_eq = theory.approx24_inclusion(block)
    assert np.allclose(p_enum, p_eq, rtol=1e-12, atol=0)
    assert math.isclose(p_eq.sum(), 2.0, rel_tol=1e-12)          # two survivors
    assert (p_eq <= 1 + 1e-12).all()
    # a_i / p_i over the pairs is unbiased, and its variance is the variance equation of Sec. 4.2
    a = np.asarray(block, dtype=np.float64)
    outcomes = []
    for i, j in itertools.permutations(range(4), 2):
        if law[i, j] == 0:
            continue
        th = np.zeros(4)
        th[i], th[j] = a[i] / p_eq[i], a[j] / p_eq[j]
        outcomes.append((law[i, j], th))
    mean, var = theory.mean_and_variance(outcomes)
    assert np.allclose(mean, a, rtol=1e-12, atol=1e-15)
    assert math.isclose(var, theory.approx24_variance(a), rel_tol=1e-10)


def test_closed_forms_on_special_blocks():
    assert np.allclose(theory.approx24_inclusion([3, 3, 3, 3]), 0.5)                 # symmetric block
    assert np.allclose(theory.approx24_inclusion([0, 5, 0, 2]), [0, 1, 0, 1])        # two non-zeros always survive
    # three equal elements and a zero: p = 2/3 each
    assert np.allclose(theory.approx24_inclusion([1, 1, 0, 1]), [2 / 3, 2 / 3, 0, 2 / 3])
    # [1, 2, 3, 4] by hand: p_4 = 4/10 + (1/10)(4/9) + (2/10)(4/8) + (3/10)(4/7)
    assert math.isclose(theory.approx24_inclusion([1, 2, 3, 4])[3], 0.4 + 4 / 90 + 0.1 + 12 / 70, rel_tol=1e-14)


def test_variance_ratio_scan_is_bounded_below_two():
    # Sec. 4.4's scan: blocks [a1, a2, a3, 1], 0 <= a1, a2, a3 <= 1; ratio of the two block variances
    grid = np.arange(0.02, 1.0 + 1e-9, 0.02)
    worst, where = 0.0, None
    for a1 in grid:
        for a2 in grid:
            for a3 in grid[::2]:
                blk = [a1, a2, a3, 1.0]
                vo = theory.opt24_variance(blk)
                if vo <= 1e-12:
                    continue
                r = theory.approx24_variance(blk) / vo
                assert r >= 1 - 1e-9                                  # never better than the optimum
                assert r < 2
                if r > worst:
                    worst, where = r, blk
    # the largest ratios sit where a_4 dominates (the scan's left edge)
    assert worst > 1.5 and max(where[:3]) <= 0.1
    # logarithmically small steps towards that edge, as the paper's footnote does (down to where
    # 1 - p_4 ~ e^2 is still well above binary64 resolution)
    for e in np.logspace(-5, -1, 30):
        for shape in ([1, 1, 1], [1, 2, 3], [1, 1e-3, 1], [1e-2, 1, 1e-1]):
            blk = [e * shape[0], e * shape[1], e * shape[2], 1.0]
            r = theory.approx24_variance(blk) / theory.opt24_variance(blk)
            assert 1 - 1e-9 <= r < 2


# ------------------------------------------------------------------ sampler vs theory ---
@pytest.mark.parametrize("block", BLOCKS + random_blocks(4))
def test_each_draw_and_the_kept_values_by_exhaustive_sweep(block):
    a32 = np.array(block, dtype=np.float32)
    a = a32.astype(np.float64)
    m = np.abs(a)
    first, second, val = oracle.sweep_approx24(a32)
    tol = 8 * 2.0 ** -24
    # first draw: |a_i| / sum
    assert np.abs(first - m / m.sum()).max() <= tol
    # second draw given the first: |a_j| / (sum - |a_i|)
    for i in range(4):
        if m[i] == 0:
            assert first[i] == 0
            continue
        want = m / (m.sum() - m[i])
        want[i] = 0
        assert np.abs(second[i] - want).max() <= tol
    # inclusion probabilities of the sampler = the equation of Sec. 4.4
    law = first[:, None] * np.nan_to_num(second)
    p_sampler = law.sum(0) + law.sum(1)
    p = theory.approx24_inclusion(a)
    assert np.abs(p_sampler - p).max() <= 4 * tol
    # survivors are a_k / p_k, and the estimator is unbiased
    nz = m > 0
    assert np.allclose(val[nz], a[nz] / p[nz], rtol=2e-6, atol=0)
    assert np.allclose(p_sampler[nz] * val[nz], a[nz], rtol=0, atol=m.sum() * 2.0 ** -20)
    # block variance from the sampler's own law = Sec. 4.2's variance equation at those p
    var = sum(p_sampler[k] * (val[k] - a[k]) ** 2 + (1 - p_sampler[k]) * a[k] ** 2 for k in range(4) if nz[k])
    assert math.isclose(var, theory.approx24_variance(a), rel_tol=1e-4, abs_tol=m.sum() ** 2 * 1e-6)


def test_worked_example_thresholds():
    # [1, 2, 3, 4]: first draw at eps = 0.1, 0.3, 0.6 changes owner; second draw among the others
    a = [1.0, 2.0, 3.0, 4.0]

    def word(eps):
        return int(eps * 2 ** 24) << 8

    def ordered(e1, e2):
        (i0, i1), _ = oracle.mvue_2of4_approx(a, word(e1), word(e2))
        return i0, i1

    assert ordered(0.05, 0.0) == (0, 1)          # first 0 (t = 0.5 < 1); others [2, 3, 4]: t = 0 -> element 1
    assert ordered(0.05, 0.3) == (0, 2)          # t2 = 2.7 in [2, 5) -> element 2
    assert ordered(0.05, 0.9) == (0, 3)          # t2 = 8.1 in [5, 9) -> element 3
    assert ordered(0.2, 0.05) == (0, 1)          # first 1 (t = 2 in [1, 3)); others [1, 3, 4]: t2 = 0.4 -> element 0
    assert ordered(0.2, 0.2) == (1, 2)           # t2 = 1.6 in [1, 4) -> element 2
    assert ordered(0.95, 0.99) == (2, 3)         # first 3; others [1, 2, 3]: t2 = 5.94 -> element 2
    # boundaries belong to the upper interval (c_k <= t)
    assert ordered(0.1, 0.0) == (0, 1)           # t = 1.0 exactly -> first is element 1, then element 0
    (_, _), (v0, v1) = oracle.mvue_2of4_approx(a, word(0.95), word(0.99))
    p = theory.approx24_inclusion(a)
    assert math.isclose(v0, 3 / p[2], rel_tol=1e-6) and math.isclose(v1, 4 / p[3], rel_tol=1e-6)


def test_zero_rules_and_signs():
    words = [0, 0xFFFFFFFF, 0x80000000, 0x12345678, 0xFFFFFF00]
    for w1, w2 in itertools.product(words, words):
        # all-zero block: positions 2 and 3 survive as (signed) zeros
        idx, val = oracle.mvue_2of4_approx([0.0, -0.0, 0.0, 0.0], w1, w2)
        assert idx == (2, 3) and val == (0.0, 0.0)
        # a lone non-zero keeps its value with a zero beside it
        for pos in range(4):
            a = [0.0] * 4
            a[pos] = -2.5
            idx, val = oracle.mvue_2of4_approx(a, w1, w2)
            assert pos in idx and idx[0] < idx[1]
            assert val[idx.index(pos)] == -2.5 and val[1 - idx.index(pos)] == 0.0
        # exactly two non-zeros: both always survive, with their own values up to binary32 rounding
        for i, j in itertools.combinations(range(4), 2):
            a = [0.0] * 4
            a[i], a[j] = 3.0, -0.125
            idx, val = oracle.mvue_2of4_approx(a, w1, w2)
            assert idx == (i, j)
            assert math.isclose(val[0], 3.0, rel_tol=4e-7) and math.isclose(val[1], -0.125, rel_tol=4e-7)
        # a zero never survives when two non-zeros exist; signs follow the source
        idx, val = oracle.mvue_2of4_approx([0.0, -1.0, 2.0, -3.0], w1, w2)
        assert 0 not in idx
        assert all(np.sign(v) == np.sign([0.0, -1.0, 2.0, -3.0][k]) for k, v in zip(idx, val))


def test_every_outcome_is_valid_on_hard_inputs():
    specials = [0.0, 1e-45, 1e-38, 1e-30, 1.0, 3.0, 1e30, 2.0 ** 100]
    words = [0, 0xFFFFFFFF, 0x7FFFFFFF, 0xFFFFFF00, 0x00000100]
    for blk in itertools.product(specials, repeat=4):
        if max(blk) / max(min(x for x in blk if x > 0) if any(blk) else 1.0, 1e-45) > 2.0 ** 126:
            continue                                     # ratios a binary32 quotient cannot hold
        for w1 in words:
            idx, val = oracle.mvue_2of4_approx(blk, w1, words[(words.index(w1) + 2) % 5])
            assert 0 <= idx[0] < idx[1] <= 3
            assert all(math.isfinite(v) for v in val)


def test_two_words_per_block_come_from_one_call_per_two_blocks():
    seed = 0x0123456789ABCDEF
    for q in (0, 1, 2, 3, 7, 2 ** 33 + 5):
        call = q >> 1
        out = oracle.philox4x32_10((call & 0xFFFFFFFF, call >> 32, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))
        assert oracle.block_word_pair(seed, q) == (out[2 * (q & 1)], out[2 * (q & 1) + 1])


def test_prune_numbers_blocks_like_per_block_calls():
    g = (RNG.standard_normal((16, 32)) * (RNG.random((16, 32)) < 0.7)).astype(np.float32)
    for axis in (0, 1):
        A = g if axis == 1 else g.T
        values, meta = oracle.prune(g, 2, 4, axis=axis, seed=11, joint=oracle.JOINT_APPROX)
        K = A.shape[1]
        for r in range(A.shape[0]):
            for j in range(K // 4):
                w1, w2 = oracle.block_word_pair(11, r * (K // 4) + j)
                idx, val = oracle.mvue_2of4_approx(A[r, 4 * j:4 * j + 4], w1, w2)
                nib = (meta[r, j // 2] >> (4 * (j % 2))) & 0xF
                assert nib == idx[0] | (idx[1] << 2)
                got = oracle.bf16_to_f32(values[r, 2 * j:2 * j + 2])
                want = oracle.bf16_to_f32(oracle.bf16_rne(np.array(val, dtype=np.float32)))
                assert np.array_equal(got, want)


# ------------------------------------------------------------------ planted mistakes ---
def _mean_with(p_wrong, a):
    law = theory.approx24_ordered_law(a)
    mean = np.zeros(4)
    for i, j in itertools.permutations(range(4), 2):
        mean[i] += law[i, j] * a[i] / p_wrong[i]
        mean[j] += law[i, j] * a[j] / p_wrong[j]
    return mean


def test_planted_mistakes_break_unbiasedness():
    a = np.array([1.0, 2.0, 3.0, 4.0])
    m = np.abs(a)
    v = m / m.sum()
    vv = v / (1 - v)
    right = v * (1 + vv.sum() - vv)
    assert np.allclose(right, theory.approx24_inclusion(a))      # Algorithm 1's v (1 + q - vv) is the same quantity
    assert np.allclose(_mean_with(right, a), a)
    assert not np.allclose(_mean_with(v * (1 + vv.sum()), a), a, rtol=1e-2)        # dropped "- vv"
    assert not np.allclose(_mean_with(2 * v, a), a, rtol=1e-2)                     # the optimal marginals instead
    assert not np.allclose(_mean_with(v, a), a, rtol=1e-2)                         # first-draw probability only
