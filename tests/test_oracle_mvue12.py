"""Pins for the oracle's MVUE 1:2 estimator against Sec. 4.1 / App. A.1."""
import math

import numpy as np
import pytest

import oracle
from oracle import theory

BLOCKS = [(1.0, 1.0), (0.25, 3.0), (-2.0, 0.5), (1e-3, -7e-3), (3.0, -3.0), (1e-20, 2e-20), (5.0, 1e-6)]


def test_closed_form_is_unbiased_with_variance_2a1a2():
    # enumeration of the two outcomes of the estimator that closes Sec. 4.1
    for a1, a2 in BLOCKS:
        mean, var = theory.mean_and_variance(theory.estimator12("mvue", a1, a2))
        assert np.allclose(mean, [a1, a2], rtol=1e-9, atol=0)
        assert math.isclose(var, theory.var12_opt(a1, a2), rel_tol=1e-9)


def test_v1_scan_has_its_minimum_at_a1_plus_a2():
    # Sec. 4.1: Var_B as a function of v_1 alone; no unbiased choice of v_1 beats a_1 + a_2
    for a1, a2 in [(1.0, 1.0), (0.3, 2.0), (4.0, 0.1)]:
        best = theory.var12_of_v1(a1, a2, a1 + a2)
        assert math.isclose(best, 2 * a1 * a2, rel_tol=1e-12)
        grid = a1 + np.geomspace(1e-4, 1e4, 20001) * a2
        vals = np.array([theory.var12_of_v1(a1, a2, v) for v in grid])
        assert vals.min() >= best * (1 - 1e-9)
        assert abs(grid[vals.argmin()] - (a1 + a2)) < 2e-3 * (a1 + a2)


@pytest.mark.parametrize("a1,a2", BLOCKS)
def test_sampler_sweep_matches_closed_form(a1, a2):
    # every one of the 2^24 values of eps through the binary32 sampler
    freq, mean, var = oracle.sweep_1of2(a1, a2)
    f1, f2 = np.float32(a1), np.float32(a2)
    p1, v1, v2 = theory.mvue12(float(f1), float(f2))
    assert abs(freq[0] - p1) <= 2.0 ** -23
    assert freq.sum() == 1.0
    scale = abs(float(f1)) + abs(float(f2))
    assert np.allclose(mean, [f1, f2], rtol=0, atol=scale * 2.0 ** -22)
    # a probability error of 2^-24 (the resolution of eps) moves the variance by about scale^2 * 2^-24
    assert math.isclose(var, theory.var12_opt(float(f1), float(f2)), rel_tol=1e-5, abs_tol=scale * scale * 2.0 ** -22)


def test_kept_value_and_threshold():
    for a1, a2 in BLOCKS:
        s = np.float32(abs(np.float32(a1))) + np.float32(abs(np.float32(a2)))
        idx, kept = oracle.mvue_1of2(a1, a2, 0)                 # eps = 0 keeps a_1 when a_1 != 0
        assert idx == 0 and kept == math.copysign(float(s), a1)
        idx, kept = oracle.mvue_1of2(a1, a2, 0xFFFFFFFF)        # eps -> 1 keeps a_2 when a_2 != 0
        assert idx == 1 and kept == math.copysign(float(s), a2)
    # threshold: keep a_1 iff eps * (|a_1| + |a_2|) < |a_1|; 1 : 3 split switches at eps = 1/4
    assert oracle.mvue_1of2(1.0, 3.0, (0x400000 - 1) << 8)[0] == 0
    assert oracle.mvue_1of2(1.0, 3.0, 0x400000 << 8)[0] == 1


def test_zero_rules():
    # a_2 = 0 always keeps a_1: a zero is never preferred to a non-zero, even when eps * S rounds up to S
    for w in (0, 0x7FFFFFFF, 0xFFFFFFFF):
        assert oracle.mvue_1of2(0.0, 0.0, w) == (0, 0.0)
        idx, kept = oracle.mvue_1of2(-0.0, -0.0, w)
        assert idx == 0 and kept == 0.0                      # a signed zero, numerically nothing
        assert oracle.mvue_1of2(0.0, -2.5, w) == (1, -2.5)
        assert oracle.mvue_1of2(2.5, 0.0, w) == (0, 2.5)
        assert oracle.mvue_1of2(-2.5, -0.0, w) == (0, -2.5)
    for n in range(0, 1 << 24, 65537):
        assert oracle.mvue_1of2(1.0, 0.0, n << 8) == (0, 1.0)
        assert oracle.mvue_1of2(0.0, 3.0, n << 8) == (1, 3.0)


def test_unit_circle_experiment():
    # Fig. 1: blocks on the first quarter of the unit circle, each sampled 100 times and
    # averaged.  For an unbiased estimator the expected squared distance of the average from
    # the block is Var_B / 100 = sin(2 phi) / 100 for MVUE (2 a_1 a_2 with a = (cos, sin)).
    phis = np.linspace(0.02, math.pi / 2 - 0.02, 400)
    q = 0
    ratio = []
    for phi in phis:
        a = (math.cos(phi), math.sin(phi))
        acc = np.zeros(2)
        for _ in range(100):
            idx, kept = oracle.mvue_1of2(a[0], a[1], oracle.block_word(77, q))
            q += 1
            acc[idx] += kept
        avg = acc / 100
        ratio.append(((avg - a) ** 2).sum() / (math.sin(2 * phi) / 100))
    # mean of 400 independent ratios with expectation 1; each ratio has variance ~2 (binomial
    # fourth moment), so 6 sigma of the mean is ~0.45
    assert abs(np.mean(ratio) - 1.0) < 0.45
    # the uniform unbiased pruner of Fig. 1(b) has spread 1/100 >= sin(2 phi)/100 everywhere
    for phi in phis[::40]:
        a1, a2 = math.cos(phi), math.sin(phi)
        _, var_u = theory.mean_and_variance(theory.estimator12("unbiased", a1, a2))
        assert math.isclose(var_u, a1 * a1 + a2 * a2, rel_tol=1e-12)
        assert var_u >= theory.var12_opt(a1, a2)


def test_negative_controls_are_rejected():
    # Table 2's other pruners: the unbiasedness check must have the power to reject them
    a1, a2 = 1.0, 3.0
    for name in ("greedy", "biased", "uniform"):
        mean, _ = theory.mean_and_variance(theory.estimator12(name, a1, a2))
        assert not np.allclose(mean, [a1, a2], rtol=1e-3)
    mean, var = theory.mean_and_variance(theory.estimator12("unbiased", a1, a2))
    assert np.allclose(mean, [a1, a2])
    assert var > theory.var12_opt(a1, a2)
