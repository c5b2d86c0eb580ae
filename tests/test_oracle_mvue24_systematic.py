"""Pins for the oracle's second 2:4 law (systematic sampling) against what Sec. 4.2 fixes:
the optimal marginals, unbiasedness and the minimal block variance; plus its zero rules,
the validity of every outcome and a worked example."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import theory

RNG = np.random.Generator(np.random.PCG64(4242))


def random_blocks(n):
    blocks = []
    for _ in range(n):
        kind = RNG.integers(0, 4)
        if kind == 0:
            a = RNG.standard_normal(4)
        elif kind == 1:
            a = np.exp(2 * RNG.standard_normal(4)) * RNG.choice([-1, 1], 4)
        elif kind == 2:
            a = RNG.standard_t(3, 4) * 1e-3
        else:
            a = RNG.standard_normal(4) * (RNG.random(4) < 0.5)
        blocks.append(a)
    return blocks


ADVERSARIAL = [
    [1, 2, 3, 4], [1, 2, 3, 5.5], [1, 1, 1, 10], [-1, 1, -1, 1], [1, 2, 3, 5],
    [1, 2, 3, 6],            # the heaviest element equals the sum of the rest: p = 1 from both criteria
    [0, 0, 3, -4], [0, 2, 0, 0], [0, 1, 1, 1], [0, 0, 0, 0], [0, 1, 2, 3],
    [1e-3, 1e3, 1.0, 1.0], [4, 3, 2, 1], [3, -1, 4, -1.5], [10, 1, 1, 1], [1, 10, 1, 1],
]
SYS = oracle.JOINT_SYSTEMATIC
HALVES = [[1, 0, 0, 1], [1, 1, 0, 0], [0, 2, 2, 0], [3, 0, 3, 0], [1, 1, 1, 3], [6, 1, 2, 3], [2, 2, 2, 2]]


def marginals_of(freq):
    marg = np.zeros(4)
    for (i, j), f in zip(oracle.PAIRS, freq):
        marg[i] += f
        marg[j] += f
    return marg


@pytest.mark.parametrize("block", ADVERSARIAL + HALVES + [list(b) for b in random_blocks(8)])
def test_sweep_has_the_optimal_marginals_mean_and_variance(block):
    a32 = np.array(block, dtype=np.float32)
    a = a32.astype(np.float64)
    freq, mean, var = oracle.sweep_2of4(a32, SYS)
    assert math.isclose(freq.sum(), 1.0, abs_tol=1e-12)
    m = np.abs(a)
    if np.count_nonzero(m) >= 2:
        # Sec. 4.2: p_i = 2 a_i / sum, or one p_i = 1 and the rest a_k / (sum of the rest)
        assert np.abs(marginals_of(freq) - theory.marginals24(m)).max() <= 8 * 2.0 ** -23
        law = theory.systematic_law24(a)
        want = np.array([law[p] for p in oracle.PAIRS])
        assert np.abs(freq - want).max() <= 8 * 2.0 ** -23
        scale = m.sum()
        assert np.allclose(mean, a, rtol=0, atol=scale * 2.0 ** -20)
        # the minimal block variance: a function of the marginals alone (variance equation of Sec. 4.2)
        want_var = theory.block_variance(m, theory.marginals24(m))
        assert math.isclose(var, want_var, rel_tol=2e-5, abs_tol=scale * scale * 1e-6)
        srt = np.sort(m)
        if srt[3] < srt[:3].sum():
            assert math.isclose(var, theory.var24_uncapped(m), rel_tol=2e-5, abs_tol=scale * scale * 1e-6)  # App. A.3
    else:
        assert freq.max() == 1.0 and np.array_equal(mean, a) and var == 0.0


@pytest.mark.parametrize("block", [[1, 2, 3, 4], [1, 2, 3, 5.5], [1, 1, 1, 10], [0, 1, 2, 3], [3, -1, 4, -1.5]])
def test_both_laws_share_marginals_and_variance(block):
    a32 = np.array(block, dtype=np.float32)
    f_tab, mean_tab, var_tab = oracle.sweep_2of4(a32, oracle.JOINT_TABLE)
    f_sys, mean_sys, var_sys = oracle.sweep_2of4(a32, SYS)
    assert np.abs(marginals_of(f_tab) - marginals_of(f_sys)).max() <= 1e-6
    assert np.allclose(mean_tab, mean_sys, rtol=0, atol=np.abs(a32).sum() * 1e-6)
    assert math.isclose(var_tab, var_sys, rel_tol=1e-5)


def test_worked_example():
    # [1,2,3,4]: D = 10, H = 5, intervals [0,1) [1,3) [3,6) [6,10); t = 5 eps, t + 5:
    # eps < 0.2 -> owners 0 and 2; 0.2 <= eps < 0.6 -> 1 and 3; else 2 and 3
    def pick(eps):
        return oracle.mvue_2of4([1, 2, 3, 4], int(eps * 2**23) << 9, SYS)
    assert pick(0.0) == ((0, 2), (5.0, 5.0))
    assert pick(0.19)[0] == (0, 2)
    assert pick(0.21)[0] == (1, 3)
    assert pick(0.59)[0] == (1, 3)
    assert pick(0.61)[0] == (2, 3)
    assert pick(0.9999999)[0] == (2, 3)
    # the block's own order matters, not the magnitudes' rank: [4,1,3,2] has intervals [0,4) [4,5) [5,8) [8,10)
    assert oracle.mvue_2of4([4, 1, 3, 2], int(0.5 * 2**23) << 9, SYS)[0] == (0, 2)     # t = 2.5, t + 5 = 7.5
    assert oracle.mvue_2of4([4, 1, 3, 2], int(0.9 * 2**23) << 9, SYS)[0] == (1, 3)     # t = 4.5, t + 5 = 9.5


def test_kept_values():
    blk = [1, -2, 3, -4]
    for w in (0, 0x12345678, 0x9ABCDEF0, 0xFFFFFFFF):
        (i0, i1), (v0, v1) = oracle.mvue_2of4(blk, w, SYS)
        assert v0 == math.copysign(5.0, blk[i0]) and v1 == math.copysign(5.0, blk[i1])   # sum / 2
    # clipped: the dominant element keeps its value, the other becomes sign * (sum of the rest)
    blk = [1, -1, -10, 1]
    seen = set()
    for w in range(0, 1 << 32, 0x01234567):
        (i0, i1), (v0, v1) = oracle.mvue_2of4(blk, w, SYS)
        kept = dict(zip((i0, i1), (v0, v1)))
        assert i0 < i1 and kept[2] == -10.0
        other = i0 if i1 == 2 else i1
        assert kept[other] == math.copysign(3.0, blk[other])
        seen.add(other)
    assert seen == {0, 1, 3}


def test_zero_rules():
    for w in (0, 1 << 9, 0x7FFFFFFF, 0x80000000, 0xFFFFFFFF):
        assert oracle.mvue_2of4([0, 0, 0, 0], w, SYS) == ((2, 3), (0.0, 0.0))
        assert oracle.mvue_2of4([-0.0, -0.0, -0.0, -0.0], w, SYS) == ((2, 3), (0.0, 0.0))
        # a lone non-zero survives with its own value, a zero next to it as a zero
        assert oracle.mvue_2of4([-2, 0, 0, 0], w, SYS) == ((0, 1), (-2.0, 0.0))
        assert oracle.mvue_2of4([0, 2, 0, 0], w, SYS) == ((1, 2), (2.0, 0.0))
        assert oracle.mvue_2of4([0, 0, 7, 0], w, SYS) == ((2, 3), (7.0, 0.0))
        assert oracle.mvue_2of4([0, 0, 0, 7], w, SYS) == ((2, 3), (0.0, 7.0))
        assert math.copysign(1.0, oracle.mvue_2of4([0, 0, -0.0, 7], w, SYS)[1][0]) == -1.0   # a signed zero
        # two non-zeros: both always survive unchanged
        assert oracle.mvue_2of4([0, 0, 3, -4], w, SYS) == ((2, 3), (3.0, -4.0))
        assert oracle.mvue_2of4([5, 0, 0, -5], w, SYS) == ((0, 3), (5.0, -5.0))
        assert oracle.mvue_2of4([0, 1e-20, 0, 3e10], w, SYS) == ((1, 3), (float(np.float32(1e-20)), float(np.float32(3e10))))
    # exactly-half intervals and empty intervals at every one of the 2^23 draws: the same two survivors
    for blk, pair in (([1, 0, 0, 1], (0, 3)), ([1, 1, 0, 0], (0, 1)), ([0, 2, 2, 0], (1, 2)), ([3, 0, 3, 0], (0, 2))):
        freq, mean, var = oracle.sweep_2of4(np.array(blk, dtype=np.float32), SYS)
        assert freq[oracle.PAIRS.index(pair)] == 1.0 and var == 0.0
    # a zero is never drawn while three non-zeros compete, at any draw
    for blk, zero in (([1, 0, 1, 1], 1), ([0, 3, 1e-3, 0.5], 0), ([2, 5, 1, 0], 3), ([1, 1, 0, 1e-6], 2)):
        freq, _, _ = oracle.sweep_2of4(np.array(blk, dtype=np.float32), SYS)
        assert marginals_of(freq)[zero] == 0.0


def test_every_outcome_is_a_valid_pair():
    rng = np.random.Generator(np.random.PCG64(77))
    blocks = [np.array(b, dtype=np.float32) for b in ADVERSARIAL + HALVES]
    for _ in range(4000):
        kind = rng.integers(0, 5)
        if kind == 0:
            a = rng.standard_normal(4)
        elif kind == 1:
            a = np.exp(8 * rng.standard_normal(4)) * rng.choice([-1, 1], 4)
        elif kind == 2:                                      # near-ties and near-half blocks
            base = rng.standard_normal()
            a = base * (1 + rng.integers(-2, 3, 4) * 2.0 ** -23)
            a[rng.integers(0, 4)] *= rng.choice([1, 2, 3])
        elif kind == 3:
            a = rng.standard_normal(4) * (rng.random(4) < 0.5)
        else:                                                # bf16-representable values, like the kernels' inputs
            a = oracle.bf16_to_f32(oracle.bf16_rne((rng.standard_normal(4) * (rng.random(4) < 0.7)).astype(np.float32)))
        blocks.append(np.asarray(a, dtype=np.float32))
    words = [0, 1 << 9, 0xFFFFFE00, 0xFFFFFFFF] + [int(x) for x in rng.integers(0, 1 << 32, 12)]
    for a in blocks:
        nz = np.flatnonzero(a)
        for w in words:
            (i, j), (vi, vj) = oracle.mvue_2of4(a, w, SYS)
            assert 0 <= i < j <= 3
            assert math.copysign(1.0, vi) == math.copysign(1.0, float(a[i]))
            assert math.copysign(1.0, vj) == math.copysign(1.0, float(a[j]))
            assert abs(vi) >= abs(float(a[i])) and abs(vj) >= abs(float(a[j]))


def test_rounding_moves_no_probability_by_more_than_the_resolution_of_eps():
    # inexact prefix sums: a clipped element is still kept, and a zero still left out, at all but
    # at most two of the 2^23 draws
    for blk in ([-1.8804901, 0.0, 0.7375498, -1.0074474], [-0.5427044, 0.0, 0.13571715, 0.0662647],
                [0.3, 0.11, 7.7, 0.05], [0.0, 1e-3, 3e-8, 7e-4], [1.1, 0.0, 0.0, 3.3], [0.7, 0.1, 0.0, 0.30000001]):
        a32 = np.array(blk, dtype=np.float32)
        freq, _, _ = oracle.sweep_2of4(a32, SYS)
        marg = marginals_of(freq)
        want = theory.marginals24(a32.astype(np.float64))
        assert np.abs(marg - want).max() <= 2 * 2.0 ** -22
        for k in range(4):
            if a32[k] == 0:
                assert marg[k] <= 2.0 ** -22
            if want[k] == 1.0:
                assert marg[k] >= 1 - 2.0 ** -22


def test_a_planted_mistake_is_caught():
    # the same sweep check applied to two wrong samplers written here: weights not clipped, and
    # the second point at t + H/2; each must break the marginals of Sec. 4.2 on some block
    def wrong_law(a, clip, step):
        m = np.abs(np.asarray(a, dtype=np.float64))
        rest = m.sum() - m
        e = np.minimum(m, rest) if clip else m
        H = e.sum() / 2
        edges = np.concatenate([[0.0], np.cumsum(e)])
        marg = np.zeros(4)
        for t in (np.arange(20000) + 0.5) / 20000 * H:
            for point in (t, t + step * H):
                marg[min(3, int(np.searchsorted(edges, point, side="right")) - 1)] += 1
        return marg / 20000
    assert np.abs(wrong_law([1, 1, 1, 10], clip=False, step=1.0) - theory.marginals24([1, 1, 1, 10])).max() > 0.05
    assert np.abs(wrong_law([1, 2, 3, 4], clip=True, step=0.5) - theory.marginals24([1, 2, 3, 4])).max() > 0.05
    assert np.abs(wrong_law([1, 2, 3, 4], clip=True, step=1.0) - theory.marginals24([1, 2, 3, 4])).max() < 1e-3
