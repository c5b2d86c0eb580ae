"""Pins for the oracle's approx-4:8 estimator (appendix "Additional sparsity results": Sec. 4.4's sequential
magnitude-proportional draws carried to four survivors of eight, kept values a_i / p_i with the exact inclusion
probability)."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import theory

RNG = np.random.Generator(np.random.PCG64(48))
BLOCKS = [
    [1, 2, 3, 4, 5, 6, 7, 8], [1, 1, 1, 1, 1, 1, 1, 1], [8, -7, 6, -5, 4, -3, 2, -1], [1e-3, 1, 1, 1, 100, 1, 1, 1],
    [0, 1, 0, 2, 3, 0, 4, 5], [0.5, 0, 0.25, 3, 0, 0.125, 1, 2],
]
BLOCKS += [list(RNG.standard_normal(8)) for _ in range(4)] + [list(RNG.standard_t(3, 8) * 1e-3) for _ in range(3)]
WORDS = (0x12345678, 0x9ABCDEF0, 0x55555555, 0xDEADBEEF)


def test_the_sequential_law_for_two_of_four_is_the_papers_equation():
    # brute force over ordered sequences against the printed inclusion probability of Sec. 4.4
    for a in ([1, 2, 3, 4], [0.3, 5, 0.01, 2], [1, 1, 1, 1], [1, 0, 2, 3]):
        assert np.allclose(theory.sequential_inclusion(a, 2), theory.approx24_inclusion(a), rtol=1e-13, atol=0)


@pytest.mark.parametrize("block", BLOCKS)
def test_inclusion_probabilities_match_brute_force(block):
    a = np.array(block, dtype=np.float32)
    _, _, p = oracle.approx_4of8(a, WORDS)
    want = theory.sequential_inclusion(a.astype(np.float64), 4)
    assert np.allclose(p, want, rtol=2e-6, atol=1e-9)
    assert math.isclose(p.sum(), 4.0, rel_tol=1e-6)
    assert (p <= 1 + 1e-6).all() and (p >= 0).all()
    # a heavier element is never less likely to survive
    order = np.argsort(np.abs(a), kind="stable")
    assert (np.diff(p[order]) >= -1e-6).all()


@pytest.mark.parametrize("block", BLOCKS)
def test_kept_values_make_the_estimator_unbiased_over_the_exact_set_law(block):
    # E[theta_i] = sum over the 70 sets of P[set] * [i in set] * value_i: with the oracle's own kept values (which do
    # not depend on the partners) this must give back a_i
    a = np.array(block, dtype=np.float32)
    value = {}
    for words in itertools.product((0x00000000, 0x3FFFFFFF, 0x7FFFFFFF, 0xBFFFFFFF, 0xFFFFFF00), repeat=4):
        idx, val, _ = oracle.approx_4of8(a, words)
        for i, v in zip(idx, val):
            assert value.setdefault(i, v) == v
    law = theory.sequential_set_law(a.astype(np.float64), 4)
    for i in range(8):
        if a[i] == 0:
            continue
        mean = sum(pr for s, pr in law.items() if i in s) * value[i]
        assert math.isclose(mean, float(a[i]), rel_tol=3e-6), (i, mean, a[i])


def test_each_draw_is_magnitude_proportional_among_the_remaining():
    # draw t, swept over 2^16 evenly spaced values of its word with the earlier words pinned: the position it adds is
    # distributed as m_k / (sum of what is left), for every one of the four draws
    a = np.array([3, 1, 4, 1, 5, 9, 2, 6], dtype=np.float32)
    m = np.abs(a).astype(np.float64)
    pinned = [0x40000000, 0xC0000000, 0x10000000]           # the earlier draws of the later sweeps
    for t in range(4):
        words = pinned[:t] + [0] * (4 - t)
        earlier = oracle.approx_4of8_order(a, words)[:t]
        counts = np.zeros(8)
        for n in range(1 << 16):
            words[t] = (n << 16) | 0x8000
            order = oracle.approx_4of8_order(a, words)
            assert order[:t] == earlier and order[t] not in earlier
            counts[order[t]] += 1
        left = m.copy()
        left[list(earlier)] = 0
        assert np.abs(counts / (1 << 16) - left / left.sum()).max() <= 3 * 2.0 ** -16, t


def test_zero_rules_and_validity():
    for w in ((0, 0, 0, 0), (0xFFFFFFFF,) * 4, WORDS):
        # at most four non-zeros: all of them survive with their own values, zeros fill up as zeros
        idx, val, _ = oracle.approx_4of8([0, 2, 0, 0, -3, 0, 0, 0], w)
        assert 1 in idx and 4 in idx and dict(zip(idx, val))[1] == 2.0 and dict(zip(idx, val))[4] == -3.0
        assert all(v == 0 for i, v in zip(idx, val) if i not in (1, 4))
        idx, val, _ = oracle.approx_4of8([1, 0, 2, 0, 3, 0, 4, 0], w)
        assert idx == (0, 2, 4, 6) and val == (1.0, 2.0, 3.0, 4.0)
        idx, val, _ = oracle.approx_4of8([0] * 8, w)
        assert len(set(idx)) == 4 and all(v == 0 for v in val)
        # more than four non-zeros: a zero is never drawn
        idx, _, _ = oracle.approx_4of8([1, 0, 2, 3, 0, 4, 5, 6], w)
        assert 1 not in idx and 4 not in idx
    # four distinct ascending positions on huge / tiny mixtures and edge words
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0**-126, 2.0**-140, 2.0**100, -2.0**110, 1e-3, 7.0], dtype=np.float32)
    for _ in range(300):
        a = pool[RNG.integers(0, len(pool), 8)]
        words = tuple(int(x) for x in RNG.integers(0, 2**32, 4))
        idx, val, _ = oracle.approx_4of8(a, words)
        assert list(idx) == sorted(set(idx)) and len(idx) == 4 and all(0 <= i < 8 for i in idx)
        # values are specified only inside the contract (non-zero magnitudes within 2^60 of each other, sums between
        # 2^-100 and 2^100: the reciprocals and their products then stay normal numbers); the pattern is always valid
        nz = np.abs(a[a != 0]).astype(np.float64)
        if nz.size == 0 or (nz.max() / nz.min() <= 2.0 ** 60 and 2.0 ** -100 <= nz.sum() <= 2.0 ** 100):
            assert all(np.isfinite(v) for v in val)
            assert all(np.sign(v) == np.sign(a[i]) or v == 0 for i, v in zip(idx, val))


def test_tensor_prune_numbering_shards_axes_and_monte_carlo():
    from paper_2203_10991_b200 import workloads
    g = workloads.gradient((64, 48), "relu_normal", seed=4, dtype="f32")
    v, mk = oracle.prune_4of8(g, 1, seed=9)
    assert v.shape == (64, 24) and mk.shape == (64, 6)
    assert all(bin(int(b)).count("1") == 4 for b in mk.ravel())
    # block numbering: block j of row r is generator call r * (K / 8) + j
    for r, j in [(0, 0), (3, 5), (63, 2)]:
        idx, val, _ = oracle.approx_4of8(g[r, 8 * j:8 * j + 8], oracle.block_words4(9, r * 6 + j))
        assert int(mk[r, j]) == sum(1 << i for i in idx)
        assert [oracle.bf16_rne(np.array([x], dtype=np.float32))[0] for x in val] == list(v[r, 4 * j:4 * j + 4])
    # axis 0 is the transposed view; K shards reproduce the unsharded run
    v0, m0 = oracle.prune_4of8(np.ascontiguousarray(g.T), 0, seed=9)
    assert np.array_equal(v0, v) and np.array_equal(m0, mk)
    vp, mp = oracle.prune_4of8(np.ascontiguousarray(g[:, 16:48]), 1, seed=9, k_total=48, k_offset=16)
    assert np.array_equal(vp, v[:, 8:]) and np.array_equal(mp, mk[:, 2:])
    # Monte Carlo over seeds: the mean of the unpacked estimate sits on g (six standard errors, bf16 storage slack)
    small = np.ascontiguousarray(g[:8, :16])
    n_seeds = 6000
    acc = np.zeros_like(small, dtype=np.float64)
    acc2 = np.zeros_like(small, dtype=np.float64)
    for seed in range(n_seeds):
        d = oracle.unpack_4of8(*oracle.prune_4of8(small, 1, seed=seed)).astype(np.float64)
        acc += d
        acc2 += d * d
    mean = acc / n_seeds
    sd = np.sqrt(np.maximum(acc2 / n_seeds - mean ** 2, 0) / n_seeds)
    assert (np.abs(mean - small) <= 6 * sd + 2.0 ** -8 * np.abs(small)).all()
    # power: the same check rejects survivors left unscaled (the biased variant of Table 2's ablation)
    kept_unscaled = np.zeros_like(small, dtype=np.float64)
    for seed in range(400):
        _, mk2 = oracle.prune_4of8(small, 1, seed=seed)
        for r in range(8):
            for j in range(2):
                for k in range(8):
                    if mk2[r, j] >> k & 1:
                        kept_unscaled[r, 8 * j + k] += small[r, 8 * j + k]
    assert np.abs(kept_unscaled / 400 - small).max() > 0.05
