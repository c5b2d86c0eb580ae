"""Pins for the oracle's stochastic rounding of survivors to bf16 (unbiased storage of a_i / p_i)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import philox_py
from paper_2203_10991_b200 import workloads


def f32(x) -> float:
    return float(np.float32(x))


def bf16_value(bits: int) -> Fraction:
    return Fraction(float(np.array([bits << 16], dtype=np.uint32).view(np.float32)[0]))


VALUES = [1.0, 1.0 + 2.0**-8, 1.0 + 2.0**-9, 1.0 + 2.0**-23, 2.0 - 2.0**-23, 3.14159274, -2.71828175, 1e-3, -7.5e5,
          2.0**-126, 2.0**-126 * (1 + 2.0**-10), 2.0**-133, 2.0**-149, -(2.0**-140), 1.9999999 * 2.0**100, 0.0, -0.0,
          0.333333343, 255.99998, -65503.996]


@pytest.mark.parametrize("x", VALUES)
def test_expectation_over_all_rounding_bits_is_exact(x):
    # exact enumeration over the 2^16 values of r, in rationals: the mean of the stored values IS x
    x = f32(x)
    total = Fraction(0)
    seen = set()
    for r in range(1 << 16):
        b = oracle.bf16_sr(x, r)
        seen.add(b)
        total += bf16_value(b)
    assert total / (1 << 16) == Fraction(x)
    # only the two neighbours on the bf16 grid ever appear, and the lower one is what truncation gives
    bits = int(np.array([x], dtype=np.float32).view(np.uint32)[0])
    lo = bits >> 16
    assert seen <= {lo, lo + 1}
    if bits & 0xFFFF == 0:
        assert seen == {lo}                                   # already on the grid: never moves
    else:
        up = sum(1 for r in range(1 << 16) if oracle.bf16_sr(x, r) == lo + 1)
        assert up == bits & 0xFFFF                            # P[up] = fraction / 2^16


def test_neighbours_bracket_the_value_and_carry_into_the_next_binade():
    for x in VALUES:
        x = f32(x)
        for r in (0, 1, 0x7FFF, 0x8000, 0xFFFF):
            v = bf16_value(oracle.bf16_sr(x, r))
            if x >= 0:
                assert bf16_value(oracle.bf16_sr(x, 0)) <= Fraction(x) <= bf16_value(oracle.bf16_sr(x, 0xFFFF))
            else:
                assert bf16_value(oracle.bf16_sr(x, 0xFFFF)) <= Fraction(x) <= bf16_value(oracle.bf16_sr(x, 0))
            assert abs(v - Fraction(x)) < abs(Fraction(x)) * Fraction(1, 128) + Fraction(1, 2**133)
    # 2 - 2^-23 rounds up to exactly 2.0 (mantissa carry) for all but one value of r
    assert oracle.bf16_sr(f32(2.0 - 2.0**-23), 0xFFFF) == 0x4000 and oracle.bf16_sr(f32(2.0 - 2.0**-23), 0) == 0x3FFF


def test_rounding_bits_are_a_generator_call_of_their_own():
    # counter (lo32(u), hi32(u), 1, 0): third word 1 keeps the stream apart from every selection draw (third word 0)
    for seed, u in [(0, 0), (7, 12345), (2**63 + 11, 2**33 + 5), (0xDEADBEEFCAFEF00D, 999)]:
        words = philox_py.philox4x32((u & 0xFFFFFFFF, u >> 32, 1, 0), (seed & 0xFFFFFFFF, seed >> 32))
        for e in range(8):
            want = (words[e >> 1] >> 16) if e & 1 else (words[e >> 1] & 0xFFFF)
            assert oracle.rounding_bits(seed, u, e) == want
        sel = philox_py.philox4x32((u & 0xFFFFFFFF, u >> 32, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))
        assert tuple(words) != tuple(sel)


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1), (2, 4, 2), (1, 4, 0)])
@pytest.mark.parametrize("axis", [0, 1])
def test_tensor_prune_with_stochastic_rounding(n, m, joint, axis):
    # same masks as round-to-nearest; every stored survivor is one of the two bf16 neighbours of the binary32 survivor
    # and equals oracle_bf16_sr with that slot's bits; bf16-exact survivors are untouched; K shards reproduce it
    g = workloads.gradient((64, 48), "relu_normal", seed=3, dtype="f32")
    g[:, ::7] *= 1.0 + 2.0**-12                                # make sure many survivors are off the bf16 grid
    v_rn, m_rn = oracle.prune(g, n, m, axis=axis, seed=5, joint=joint)
    v_sr, m_sr = oracle.prune(g, n, m, axis=axis, seed=5, joint=joint, stochastic_rounding=True)
    assert np.array_equal(m_rn, m_sr)
    diff = v_sr.astype(np.int32) - v_rn.astype(np.int32)
    assert set(np.unique(diff)) <= {-1, 0, 1} and np.count_nonzero(diff) > 0
    K = g.shape[1] if axis == 1 else g.shape[0]
    lo, hi = 16, 48 if axis == 1 else 64
    part = np.ascontiguousarray(g[:, lo:hi] if axis == 1 else g[lo:hi])
    v_p, m_p = oracle.prune(part, n, m, axis=axis, seed=5, joint=joint, stochastic_rounding=True, k_total=K, k_offset=lo)
    assert np.array_equal(v_p, v_sr[:, lo // 2:hi // 2]) and np.array_equal(m_p, m_sr[:, lo // 8:hi // 8])
    # a different seed rounds differently (same masks would need the same selection words too, so compare values only)
    v_sr2, _ = oracle.prune(g, n, m, axis=axis, seed=6, joint=joint, stochastic_rounding=True)
    assert not np.array_equal(v_sr, v_sr2)


def test_slot_numbering_of_the_tensor_prune():
    # one row of A, K = 32 (two units): recompute every stored survivor from the round-to-nearest run's masks, the
    # block samplers and the slot's bits
    g = (np.arange(1, 33, dtype=np.float32) * np.float32(1.0 + 2.0**-11)).reshape(1, 32)
    seed = 99
    v_sr, meta = oracle.prune(g, 2, 4, axis=1, seed=seed, joint=1, stochastic_rounding=True)
    for j in range(8):
        idx, val = oracle.mvue_2of4(g[0, 4 * j:4 * j + 4], oracle.block_word(seed, j), joint=1)
        for e in range(2):
            want = oracle.bf16_sr(val[e], oracle.rounding_bits(seed, j // 4, 2 * (j % 4) + e))
            assert int(v_sr[0, 2 * j + e]) == want


def test_mean_over_seeds_has_no_storage_bias():
    # a block whose survivor value S/2 sits 1/4 of the way between two bf16 numbers: with round-to-nearest every
    # stored survivor is the lower neighbour (relative bias 2^-10 on E[theta]); with stochastic rounding the
    # mean over seeds converges on the block itself
    a = np.array([[1.0, 1.0, 1.0, 1.0 + 2.0**-6] * 4], dtype=np.float32)      # S/2 = 2 + 2^-7 -> between 2.0 and 2.015625
    n_seeds = 4000
    acc_rn = np.zeros(16)
    acc_sr = np.zeros(16)
    for seed in range(n_seeds):
        v, mt = oracle.prune(a, 2, 4, axis=1, seed=seed, joint=1)
        acc_rn += oracle.unpack(v, mt)[0]
        v, mt = oracle.prune(a, 2, 4, axis=1, seed=seed, joint=1, stochastic_rounding=True)
        acc_sr += oracle.unpack(v, mt)[0]
    total = float(a.sum())
    # sum over the block of E[theta_i] = sum a_i; storage rounding shifts it by S/2 -> 2.0, i.e. by a factor 2 / (2 + 2^-7)
    assert abs(acc_rn.sum() / n_seeds - total * 2.0 / (2.0 + 2.0**-7)) < 1e-9
    sd = np.sqrt(16 * (2.0**-7 * 0.5) ** 2 / n_seeds) * 2                       # rounding noise only (the masks' sum is fixed)
    assert abs(acc_sr.sum() / n_seeds - total) < 6 * sd
    assert abs(acc_rn.sum() / n_seeds - total) > 20 * sd
