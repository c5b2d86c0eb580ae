"""Pins for the oracle's MVUE 1:4 sampler: the keep-one estimator of Sec. 4.1 on a block of four (the MVUE 1:4 of
the appendix "Additional sparsity results")."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import theory

RNG = np.random.Generator(np.random.PCG64(14))
BLOCKS = [[1, 2, 3, 4], [4, 3, 2, 1], [1, 1, 1, 10], [-1, 1, -1, 1], [0, 1, 2, 3], [0, 0, 3, -4], [0, 2, 0, 0],
          [1e-3, 1e3, 1.0, 1.0], [3, -1, 4, -1.5], [2, 2, 2, 2]] + [list(RNG.standard_normal(4)) for _ in range(4)] + \
         [list(np.exp(2 * RNG.standard_normal(4)) * RNG.choice([-1, 1], 4)) for _ in range(4)]


@pytest.mark.parametrize("block", BLOCKS)
def test_exhaustive_sweep_gives_the_law_the_mean_and_the_minimal_variance(block):
    a32 = np.array(block, dtype=np.float32)
    a = a32.astype(np.float64)
    m = np.abs(a)
    freq, mean, var = oracle.sweep_1of4(a32)
    assert math.isclose(freq.sum(), 1.0, abs_tol=1e-12)
    assert np.abs(freq - m / m.sum()).max() <= 4 * 2.0 ** -24                       # p_i = |a_i| / S
    assert np.allclose(mean, a, rtol=0, atol=m.sum() * 2.0 ** -20)                   # unbiased
    assert math.isclose(var, theory.var1m_opt(a), rel_tol=1e-5, abs_tol=m.sum() ** 2 * 1e-6)


def test_variance_closed_form_is_the_minimum_over_the_simplex_and_reduces_to_sec_4_1():
    a = np.array([1.0, 2.0, 3.0, 4.0])
    best = theory.var1m_opt(a)
    assert math.isclose(best, 100.0 - 30.0)
    assert math.isclose(theory.var1m_of_p(a, a / a.sum()), best)
    grid = np.linspace(0.02, 0.94, 24)
    for p1, p2, p3 in itertools.product(grid, repeat=3):                             # brute force over probabilities
        p4 = 1.0 - p1 - p2 - p3
        if p4 <= 0.01:
            continue
        assert theory.var1m_of_p(a, [p1, p2, p3, p4]) >= best - 1e-9
    # a block of two: the same formula is Sec. 4.1's 2 |a_1| |a_2|
    for a1, a2 in [(1.0, 2.0), (-3.0, 0.5), (7.0, 7.0)]:
        assert math.isclose(theory.var1m_opt([a1, a2]), theory.var12_opt(a1, a2))
    # the uniform keep-one estimator (p = 1/4, value 4 a_i) is unbiased too and strictly worse
    assert theory.var1m_of_p(a, [0.25] * 4) > best


def test_with_two_zeros_it_is_the_one_of_two_sampler():
    # [a, b, 0, 0]: same running sums, same threshold, same survivor and value as MVUE 1:2 on (a, b)
    for a, b in [(1.0, 2.0), (-3.0, 0.5), (1e-3, 7.0)]:
        for word in (0, 0x12345678, 0x80000000, 0xFFFFFFFF, 0x55555500):
            i4, v4 = oracle.mvue_1of4([a, b, 0.0, 0.0], word)
            i2, v2 = oracle.mvue_1of2(a, b, word)
            assert (i4, v4) == (i2, v2)


def test_thresholds_zero_rules_and_signs():
    a = [1.0, -1.0, 2.0, -4.0]                                   # S = 8: boundaries at eps = 1/8, 2/8, 4/8, all exact

    def word(eps):
        return int(eps * 2 ** 24) << 8

    assert oracle.mvue_1of4(a, word(0.0625)) == (0, 8.0)         # t = 0.5 in [0, 1)
    assert oracle.mvue_1of4(a, word(0.125)) == (1, -8.0)         # t = 1.0: boundaries belong to the upper interval
    assert oracle.mvue_1of4(a, word(0.125) - 0x100) == (0, 8.0)  # one step below it
    assert oracle.mvue_1of4(a, word(0.25)) == (2, 8.0)
    assert oracle.mvue_1of4(a, word(0.4999)) == (2, 8.0)
    assert oracle.mvue_1of4(a, word(0.5)) == (3, -8.0)
    assert oracle.mvue_1of4(a, 0xFFFFFFFF) == (3, -8.0)
    for w in (0, 0xFFFFFFFF, 0x80000000):
        assert oracle.mvue_1of4([0.0, 0.0, 0.0, -0.0], w)[0] == 3            # all-zero block keeps its last element
        for pos in range(4):
            blk = [0.0] * 4
            blk[pos] = -2.5
            assert oracle.mvue_1of4(blk, w) == (pos, -2.5)                    # a lone non-zero always survives, unchanged
        i, v = oracle.mvue_1of4([0.0, 5.0, 0.0, 1.0], w)
        assert i in (1, 3) and abs(v) == 6.0                                  # zeros are never drawn


def test_prune_stores_the_survivor_beside_a_zero_in_the_2of4_container():
    g = (RNG.standard_normal((16, 32)) * (RNG.random((16, 32)) < 0.7)).astype(np.float32)
    for axis in (0, 1):
        A = g if axis == 1 else g.T
        values, meta = oracle.prune(g, 1, 4, axis=axis, seed=21)
        K = A.shape[1]
        dense = oracle.unpack(values, meta)
        for r in range(A.shape[0]):
            for j in range(K // 4):
                i, v = oracle.mvue_1of4(A[r, 4 * j:4 * j + 4], oracle.block_word(21, r * (K // 4) + j))
                nib = (meta[r, j // 2] >> (4 * (j % 2))) & 0xF
                assert nib == ((i | (3 << 2)) if i < 3 else (2 | (3 << 2)))
                want = np.zeros(4, dtype=np.float32)
                want[i] = oracle.bf16_to_f32(oracle.bf16_rne(np.array([v], dtype=np.float32)))[0]
                assert np.array_equal(dense[r, 4 * j:4 * j + 4], want)
    # K shards reproduce the unsharded masks
    v_all, m_all = oracle.prune(g, 1, 4, axis=1, seed=21)
    v_p, m_p = oracle.prune(np.ascontiguousarray(g[:, 16:]), 1, 4, axis=1, seed=21, k_total=32, k_offset=16)
    assert np.array_equal(v_p, v_all[:, 8:]) and np.array_equal(m_p, m_all[:, 2:])
