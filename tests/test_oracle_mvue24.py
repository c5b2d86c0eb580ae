"""Pins for the oracle's MVUE 2:4 estimator against Sec. 4.2, 4.3 and App. A.2 / A.3."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import theory

RNG = np.random.Generator(np.random.PCG64(2024))


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
    [1, 2, 3, 4], [1, 2, 3, 5.5], [1, 1, 1, 10], [-1, 1, -1, 1],
    [1, 2, 3, 5],            # boundary case 1 / case 2: a_4 = 2 a_1 + a_3
    [1, 2, 3, 6],            # boundary case 2 / case 3: a_4 = a_1 + a_2 + a_3
    [0, 0, 3, -4], [0, 2, 0, 0], [0, 1, 1, 1], [0, 0, 0, 0], [2, 2, 2, 2], [0, 1, 2, 3],
    [1e-3, 1e3, 1.0, 1.0], [4, 3, 2, 1], [3, -1, 4, -1.5],
]


# ----------------------------------------------------------- theory -------
def test_pair_table_is_a_law_with_the_optimal_marginals():
    # App. A.2: every p_ij in [0,1], sum 1, row sums = the marginals of Sec. 4.2
    for a in random_blocks(3000) + [np.array(b, dtype=float) for b in ADVERSARIAL]:
        m = np.sort(np.abs(a))
        if m[3] == 0 or m[0] + m[1] + m[2] == 0:
            continue
        table = theory.pair_table24(m)
        probs = np.array(list(table.values()))
        assert (probs >= -1e-12).all() and (probs <= 1 + 1e-12).all()
        assert math.isclose(probs.sum(), 1.0, rel_tol=0, abs_tol=1e-12)
        marg = np.zeros(4)
        for (i, j), p in table.items():
            marg[i - 1] += p
            marg[j - 1] += p
        assert np.allclose(marg, theory.marginals24(m), rtol=0, atol=1e-12)
        # the worked check of App. A.2: p_1 / p_2 = a_1 / a_2
        if m[1] > 0 and m[3] < m[0] + m[1] + m[2]:
            assert math.isclose(marg[0] / marg[1], m[0] / m[1], rel_tol=1e-9, abs_tol=1e-12)


def test_cases_agree_on_their_boundaries():
    for a1, a2, a3 in [(1, 2, 3), (0.5, 0.7, 2.0), (1, 1, 1)]:
        b12 = 2 * a1 + a3
        lo = theory.pair_table24([a1, a2, a3, b12 * (1 - 1e-13)])
        hi = theory.pair_table24([a1, a2, a3, b12 * (1 + 1e-13)])
        assert all(abs(lo[k] - hi[k]) < 1e-11 for k in lo)
        b23 = a1 + a2 + a3
        lo = theory.pair_table24([a1, a2, a3, b23 * (1 - 1e-13)])
        hi = theory.pair_table24([a1, a2, a3, b23 * (1 + 1e-13)])
        assert all(abs(lo[k] - hi[k]) < 1e-11 for k in lo)


def test_marginals_satisfy_the_optimality_conditions():
    # Sec. 4.2: either p_i = 2 a_i / sum for all i, or one p_i = 1 and p_k = a_k / sum_{j != i} a_j
    for a in random_blocks(2000):
        m = np.abs(a)
        if np.count_nonzero(m) < 2:
            continue
        p = theory.marginals24(m)
        assert math.isclose(p.sum(), 2.0, rel_tol=1e-12)
        assert (p <= 1 + 1e-12).all() and (p >= 0).all()
        if p.max() < 1:
            assert np.allclose(p, 2 * m / m.sum())
        else:
            i = int(np.argmax(m))
            rest = m.sum() - m[i]
            assert p[i] == 1.0
            assert np.allclose(np.delete(p, i), np.delete(m, i) / rest)


def test_no_feasible_marginal_beats_the_optimum():
    # brute force over random feasible p (sum 2, 0 < p_i <= 1) and local perturbations
    for a in random_blocks(60) + [np.array(b, dtype=float) for b in ADVERSARIAL]:
        m = np.abs(a)
        if np.count_nonzero(m) < 3:
            continue
        p_star = theory.marginals24(m)
        best = theory.block_variance(m, p_star)
        cand = RNG.dirichlet(np.ones(4), 4000) * 2
        cand = cand[(cand <= 1).all(1) & (cand > 1e-9).all(1)]
        local = p_star + 1e-3 * RNG.standard_normal((2000, 4))
        local -= (local.sum(1, keepdims=True) - 2) / 4
        local = local[(local <= 1).all(1) & (local > 1e-9).all(1)]
        for p in np.vstack([cand, local]):
            assert theory.block_variance(m, p) >= best * (1 - 1e-9) - 1e-300


def test_variance_closed_forms_and_the_1of2_inequality():
    for a in random_blocks(2000):
        m = np.sort(np.abs(a))
        if m[2] == 0:
            continue
        v = theory.block_variance(m, theory.marginals24(m))
        if m[3] < m[0] + m[1] + m[2]:
            assert math.isclose(v, theory.var24_uncapped(m), rel_tol=1e-9, abs_tol=1e-15 * float(m[3]) ** 2)   # App. A.3
        else:
            s3 = m[0] + m[1] + m[2]
            assert math.isclose(v, s3 * s3 - (m[:3] ** 2).sum(), rel_tol=1e-9, abs_tol=1e-15 * float(m[3]) ** 2)
        # Sec. 4.3: one 2:4 block never has more variance than two 1:2 blocks, in any arrangement
        for perm in itertools.permutations(range(4)):
            b = np.abs(a)[list(perm)]
            assert v <= theory.var12_opt(b[0], b[1]) + theory.var12_opt(b[2], b[3]) + 1e-12 * (1 + v)


# ----------------------------------------------------------- sampler -------
@pytest.mark.parametrize("block", ADVERSARIAL + [list(b) for b in random_blocks(6)])
def test_sampler_sweep_matches_the_table(block):
    a32 = np.array(block, dtype=np.float32)
    a = a32.astype(np.float64)
    freq, mean, var = oracle.sweep_2of4(a32)
    assert math.isclose(freq.sum(), 1.0, abs_tol=1e-12)
    m = np.abs(a)
    nnz = np.count_nonzero(m)
    if nnz >= 2:
        law = theory.outcome_law24(a)
        want = np.array([law[p] for p in oracle.PAIRS])
        # 24-bit eps: each threshold is off by at most 2^-24 plus binary32 rounding of the walk
        assert np.abs(freq - want).max() <= 6 * 2.0 ** -24
        scale = m.sum()
        assert np.allclose(mean, a, rtol=0, atol=scale * 2.0 ** -21)
        want_var = theory.block_variance(m, theory.marginals24(m))
        assert math.isclose(var, want_var, rel_tol=2e-5, abs_tol=scale * scale * 1e-6)
    else:
        # fewer than two non-zeros: deterministic, exact, zero variance
        assert freq.max() == 1.0 and np.array_equal(mean, a) and var == 0.0


def test_kept_values():
    # uncapped: both survivors become sign(a_i) * sum / 2
    (i0, i1), (v0, v1) = oracle.mvue_2of4([1, -2, 3, -4], 0x12345678)
    assert {abs(v0), abs(v1)} == {5.0}
    assert v0 == math.copysign(5.0, [1, -2, 3, -4][i0]) and v1 == math.copysign(5.0, [1, -2, 3, -4][i1])
    # capped: the dominant element is kept unchanged, the other becomes sign * (sum of the rest)
    for w in (0, 0x55555555, 0xAAAAAAAA, 0xFFFFFFFF):
        (i0, i1), (v0, v1) = oracle.mvue_2of4([1, -1, -10, 1], w)
        assert 2 in (i0, i1) and i0 < i1
        kept = dict(zip((i0, i1), (v0, v1)))
        assert kept[2] == -10.0
        other = i0 if i1 == 2 else i1
        assert kept[other] == math.copysign(3.0, [1, -1, -10, 1][other])


def test_walk_order_and_thresholds():
    # [1,2,3,4]: denominators 2*10; cumulative numerators 13:1, 14:3, 23:3, 24:5, then 34:8
    # => eps thresholds 0.05, 0.20, 0.35, 0.60
    def pick(eps):
        return oracle.mvue_2of4([1, 2, 3, 4], int(eps * 2**24) << 8)[0]
    assert pick(0.02) == (0, 2)
    assert pick(0.10) == (0, 3)
    assert pick(0.30) == (1, 2)
    assert pick(0.50) == (1, 3)
    assert pick(0.70) == (2, 3)
    # a permuted block reports original positions, ascending
    assert oracle.mvue_2of4([4, 1, 3, 2], int(0.02 * 2**24) << 8)[0] == (1, 2)      # sorted pair 13
    assert oracle.mvue_2of4([4, 1, 3, 2], int(0.10 * 2**24) << 8)[0] == (0, 1)      # sorted pair 14


def test_zero_and_tie_rules():
    # zeros have zero-width intervals in the walk: they survive only when fewer than two non-zeros
    # exist, as the top ranks of the (magnitude, position) order, with value zero
    for w in (0, 0x7FFFFFFF, 0xFFFFFFFF):
        assert oracle.mvue_2of4([0, 0, 0, 0], w) == ((2, 3), (0.0, 0.0))
        assert oracle.mvue_2of4([-0.0, -0.0, -0.0, -0.0], w) == ((2, 3), (0.0, 0.0))
        assert oracle.mvue_2of4([0, 2, 0, 0], w) == ((1, 3), (2.0, 0.0))
        assert oracle.mvue_2of4([-2, 0, 0, 0], w) == ((0, 3), (-2.0, 0.0))
        assert oracle.mvue_2of4([0, 0, 0, 7], w) == ((2, 3), (0.0, 7.0))
        # two non-zeros: both always survive, unchanged in expectation AND in value
        (idx, val) = oracle.mvue_2of4([0, 0, 3, -4], w)
        assert idx == (2, 3) and val == (3.0, -4.0)
        (idx, val) = oracle.mvue_2of4([5, 0, 0, -5], w)
        assert idx == (0, 3) and val == (5.0, -5.0)
    # a zero is never chosen while three non-zeros compete for two slots
    for n in range(0, 1 << 24, 4099):
        idx, _ = oracle.mvue_2of4([1, 0, 1, 1], n << 8)
        assert 1 not in idx
        idx, _ = oracle.mvue_2of4([0, 3, 1e-3, 0.5], n << 8)
        assert 0 not in idx
    # ties are ordered by position: [2,2,2,2] sorts as positions 0,1,2,3
    law = theory.outcome_law24([2, 2, 2, 2])
    assert law[(0, 1)] == 0.0 and math.isclose(law[(2, 3)], 0.0, abs_tol=1e-15)
    freq, _, _ = oracle.sweep_2of4(np.array([2, 2, 2, 2], dtype=np.float32))
    assert freq[0] == 0.0 and freq[5] <= 2.0 ** -23


def test_case3_keeps_the_dominant_element_for_every_eps():
    # the dominant element survives for all 2^24 values of eps, also on the case 2 / case 3 boundary
    for block in ([1, 2, 3, 6], [1, 1, 1, 10], [0.3, 0.1, 7.0, 0.2], [1e-3, 1e-3, 1e-3, 3e-3]):
        freq, mean, _ = oracle.sweep_2of4(np.array(block, dtype=np.float32))
        top = int(np.argmax(np.abs(block)))
        with_top = sum(f for (pair, f) in zip(oracle.PAIRS, freq) if top in pair)
        assert with_top == 1.0
        assert mean[top] == np.float32(block[top])


# ------------------------------------------- the appendix, case by case -------
# oracle.mvue_2of4_cases is App. A.2 as printed (three branches, each with its own numerators and denominator,
# divisions, binary64); oracle.mvue_2of4 is the binary32, division-free evaluation that the GPU reproduces.
CASE_BLOCKS = [b for b in ADVERSARIAL if np.count_nonzero(b) >= 2] + [list(b) for b in random_blocks(10)]
PAIR_SLIPS_PER_BLOCK = 4          # draws (of 2^24) on which binary32 rounding of a threshold may move the pair (seen: <= 2)


@pytest.mark.parametrize("block", CASE_BLOCKS)
def test_binary32_sampler_equals_the_case_by_case_appendix(block):
    a32 = np.array(block, dtype=np.float32)
    if np.count_nonzero(a32) < 2:
        pytest.skip("fewer than two non-zeros: outside the appendix (zero rule)")
    which, slips, rel = oracle.sweep_2of4_cases(a32)
    m = np.sort(np.abs(a32.astype(np.float64)))
    want_case = 3 if m[3] >= m[0] + m[1] + m[2] else (1 if m[3] <= 2 * m[0] + m[2] else 2)
    assert which == want_case
    # same pair on every draw but a handful, same kept values to binary32 rounding on all of them
    assert slips <= PAIR_SLIPS_PER_BLOCK
    assert rel <= 2.0 ** -22           # three binary32 additions against exact binary64 (seen: 2^-24.2)


def test_case_by_case_appendix_on_single_draws():
    # [1,2,3,4] is case 1 with denominators 2 * 10: p_13 = 1/20, p_14 = 3/20, p_23 = 3/20, p_24 = 5/20, p_34 = 8/20
    def pick(eps):
        return oracle.mvue_2of4_cases([1, 2, 3, 4], int(eps * 2**24) << 8)
    assert pick(0.02)[:2] == (1, (0, 2)) and pick(0.10)[:2] == (1, (0, 3)) and pick(0.30)[:2] == (1, (1, 2))
    assert pick(0.50)[:2] == (1, (1, 3)) and pick(0.70)[:2] == (1, (2, 3))
    assert np.allclose(pick(0.30)[2], (5.0, 5.0), rtol=1e-15)                 # a_i / p_i = sum / 2
    # case 2, [1,2,3,5.5] (sum 11.5): p_14 = 2/11.5, p_23 = 0.5/11.5, p_24 = 3.5/11.5, p_34 = 5.5/11.5
    which, idx, val = oracle.mvue_2of4_cases([1, 2, 3, 5.5], int(0.1 * 2**24) << 8)
    assert (which, idx) == (2, (0, 3)) and np.allclose(val, (5.75, 5.75), rtol=1e-15)
    assert oracle.mvue_2of4_cases([1, 2, 3, 5.5], int(0.2 * 2**24) << 8)[1] == (1, 2)
    # case 3, [1,-1,-10,1]: the dominant element keeps its value, the partner becomes sign * 3
    which, idx, val = oracle.mvue_2of4_cases([1, -1, -10, 1], int(0.5 * 2**24) << 8)
    assert which == 3 and idx == (1, 2) and np.allclose(val, (-3.0, -10.0), rtol=1e-15)
    # fewer than two non-zeros: the appendix has nothing to say (0/0)
    assert oracle.mvue_2of4_cases([0, 2, 0, 0], 0)[0] == -1
    assert oracle.mvue_2of4_cases([0, 0, 0, 0], 0)[0] == -1


def test_the_comparison_with_the_appendix_has_power():
    # one mistake planted in each case of the case-by-case statement: the sweep then disagrees with the binary32
    # sampler on a macroscopic share of the draws, not on a handful
    for mistake, block in ((1, [1, 2, 3, 4]), (2, [1, 2, 3, 5.5]), (3, [1, 2, 3, 10])):
        a32 = np.array(block, dtype=np.float32)
        which, slips, _ = oracle.sweep_2of4_cases(a32, mistake)
        assert which == mistake
        assert slips > 2 ** 24 // 50
        assert oracle.sweep_2of4_cases(a32)[1] <= PAIR_SLIPS_PER_BLOCK


@pytest.mark.parametrize("joint", [oracle.JOINT_TABLE, oracle.JOINT_SYSTEMATIC])
@pytest.mark.parametrize("dist,seed", [("student_t", 3), ("relu_lognormal", 4), ("tile", 5)])
def test_survivors_are_their_own_value_or_one_common_raised_value(joint, dist, seed):
    """Sec. 4.2: a survivor becomes a_i / p_i, which is one common magnitude (half the clipped sum) for every survivor
    with p_i < 1 and the element itself when p_i = 1.  So in every bf16 block, with H = the smaller of the two stored
    magnitudes, each survivor stores max(|a_i|, H), with its own sign: no stored value is below its element, and two
    survivors that were both raised store the same magnitude.  (The CUDA kernels gather the survivors by position and
    raise them with one maximum against the rounded common value; this is the property that makes that exact.)"""
    from paper_2203_10991_b200 import workloads as gen
    rows, K = 256, 512
    if dist == "tile":      # adversarial blocks: ties, zeros, dominant elements, neighbours in bf16, tiny and huge scales
        pats = np.array([[1, 1, 1, 1], [0, 0, 0, 3], [0, 2, 0, 0], [1, 2, 3, 7], [1, 2, 3, 6], [1, 2, 3, 5.96875],
                         [1, 1.0078125, 1, 1.0078125], [0, 0, 5, 5], [1e-38, 2e-38, 3e-38, 1e-37],
                         [3e38, 1e38, 2e38, 3e38], [0, 0, 0, 0], [1, -1, 1, -1], [-4, 1, 0.5, 0.25],
                         [2 ** -126, 2 ** -127, 2 ** -130, 2 ** -133], [7, 0, 0, 7], [1, 255, 256, 257]], dtype=np.float32)
        g32 = np.tile(pats.reshape(-1), rows * K // pats.size + 1)[:rows * K].reshape(rows, K)
        g = oracle.bf16_rne(g32[:1]).repeat(rows, axis=0)                     # every pattern is a bf16 number already
    else:
        g = gen.gradient((rows, K), dist, seed, dtype="bf16")
    values, meta = oracle.prune(g, 2, 4, axis=1, seed=seed, joint=joint)
    a = (g & 0x7FFF).astype(np.int64).reshape(rows, K // 4, 4)              # magnitudes as ordered integers
    nib = np.stack([meta & 15, meta >> 4], axis=-1).reshape(rows, K // 4)   # block j: low nibble first
    i0, i1 = nib & 3, nib >> 2
    assert (i0 < i1).all()
    v = values.reshape(rows, K // 4, 2)
    own = np.stack([np.take_along_axis(a, i0[..., None], 2)[..., 0], np.take_along_axis(a, i1[..., None], 2)[..., 0]], -1)
    sign_in = np.stack([np.take_along_axis(g.reshape(rows, K // 4, 4), i0[..., None], 2)[..., 0],
                        np.take_along_axis(g.reshape(rows, K // 4, 4), i1[..., None], 2)[..., 0]], -1) & 0x8000
    out = (v & 0x7FFF).astype(np.int64)
    assert ((v & 0x8000) == sign_in).all()
    H = out.min(axis=-1, keepdims=True)
    assert (out == np.maximum(own, H)).all()
    assert (out != own).any() and (out == own).any()                        # both kinds occur in the sample
