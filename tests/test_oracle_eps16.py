"""Pins for the sixteen-bits-per-block random stream (one generator call per eight blocks): where the bits come from,
that the block samplers see them as an ordinary word, what resolution the probabilities keep, and that the estimators
stay unbiased to that resolution."""
import math

import numpy as np
import pytest

import oracle
from oracle import philox_py, theory
from paper_2203_10991_b200 import workloads


def test_bits_are_the_halves_of_one_call_per_eight_blocks():
    for seed in (0, 7, 2**63 + 11):
        for q in (0, 1, 2, 7, 8, 13, 2**35 + 5, 2**35 + 6):
            call = q >> 3
            words = philox_py.philox4x32((call & 0xFFFFFFFF, call >> 32, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))
            w = words[(q >> 1) & 3]
            half = (w >> 16) if q & 1 else (w & 0xFFFF)
            assert oracle.block_word16(seed, q) == half << 16
        for q in (0, 1, 3, 4, 2**34 + 2):
            call = q >> 2
            w = philox_py.philox4x32((call & 0xFFFFFFFF, call >> 32, 0, 0), (seed & 0xFFFFFFFF, seed >> 32))[q & 3]
            assert oracle.block_word_pair16(seed, q) == ((w & 0xFFFF) << 16, w & 0xFFFF0000)
    # the sixteen-bit values of consecutive blocks are uniform and uncorrelated (chi-square on 2^6 bins, lag-1 correlation)
    vals = np.array([oracle.block_word16(3, q) >> 16 for q in range(1 << 16)], dtype=np.float64)
    counts = np.bincount((vals // 1024).astype(int), minlength=64)
    chi2 = ((counts - 1024.0) ** 2 / 1024.0).sum()
    assert chi2 < 63 + 6 * math.sqrt(2 * 63)
    x = vals / 65536.0 - 0.5
    assert abs((x[:-1] * x[1:]).mean() / x.var()) < 6 / math.sqrt(len(x))


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1), (2, 4, 2), (1, 4, 0)])
def test_tensor_prune_uses_the_block_samplers_unchanged(n, m, joint):
    g = workloads.gradient((8, 64), "relu_normal", seed=2, dtype="f32")
    seed = 21
    v, mt = oracle.prune(g, n, m, axis=1, seed=seed, joint=joint, eps16=True)
    for r in (0, 5):
        for j in range(16):
            a = g[r, 4 * j:4 * j + 4]
            if m == 2:
                kept = []
                for half in range(2):
                    q = r * 32 + 2 * j + half
                    idx, val = oracle.mvue_1of2(a[2 * half], a[2 * half + 1], oracle.block_word16(seed, q))
                    kept.append((2 * half + idx, val))
                want_idx, want_val = (kept[0][0], kept[1][0]), (kept[0][1], kept[1][1])
            else:
                q = r * 16 + j
                if n == 1:
                    i, val = oracle.mvue_1of4(a, oracle.block_word16(seed, q))
                    want_idx, want_val = ((i, 3), (val, 0.0)) if i < 3 else ((2, 3), (0.0, val))
                elif joint == 2:
                    want_idx, want_val = oracle.mvue_2of4_approx(a, *oracle.block_word_pair16(seed, q))
                else:
                    want_idx, want_val = oracle.mvue_2of4(a, oracle.block_word16(seed, q), joint=joint)
            byte = mt[r, j // 2]
            nib = (byte >> 4) if j % 2 else (byte & 15)
            assert (nib & 3, nib >> 2) == tuple(want_idx)
            assert list(v[r, 2 * j:2 * j + 2]) == [oracle.bf16_rne(np.array([x], dtype=np.float32))[0] for x in want_val]
    # K shards and the transposed view agree with the whole tensor, as for the 32-bit stream
    vp, mp = oracle.prune(np.ascontiguousarray(g[:, 32:]), n, m, axis=1, seed=seed, joint=joint, eps16=True,
                          k_total=64, k_offset=32)
    assert np.array_equal(vp, v[:, 16:]) and np.array_equal(mp, mt[:, 4:])
    v0, m0 = oracle.prune(np.ascontiguousarray(g.T), n, m, axis=0, seed=seed, joint=joint, eps16=True)
    assert np.array_equal(v0, v) and np.array_equal(m0, mt)


def test_probabilities_keep_a_resolution_of_two_to_the_minus_sixteen():
    # all 2^16 values of the block's bits through the unchanged samplers: outcome frequencies within a few 2^-16 of
    # the laws that the 2^24 sweeps pin exactly, means within that resolution of the block
    for block in ([1, 2, 3, 4], [1, 2, 3, 5.5], [1, 1, 1, 10], [0.3, -0.1, 4.0, -1.5], [0, 1, 2, 3]):
        a = np.array(block, dtype=np.float32)
        m = np.abs(a.astype(np.float64))
        for joint, law_fn, slack in ((0, theory.outcome_law24, 8), (1, theory.systematic_law24, 16)):
            counts = {p: 0 for p in oracle.PAIRS}
            mean = np.zeros(4)
            for h in range(1 << 16):
                idx, val = oracle.mvue_2of4(a, h << 16, joint=joint)
                counts[idx] += 1
                mean[list(idx)] += val
            law = law_fn(a.astype(np.float64))
            for pair in oracle.PAIRS:
                assert abs(counts[pair] / 65536.0 - law[pair]) <= slack * 2.0 ** -16, (block, joint, pair)
            assert np.abs(mean / 65536.0 - a).max() <= slack * 2.0 ** -16 * m.sum()
    for a1, a2 in ((1.0, 3.0), (0.2, 0.1), (5.0, 1e-3)):
        keep1 = sum(1 for h in range(1 << 16) if oracle.mvue_1of2(a1, a2, h << 16)[0] == 0)
        assert abs(keep1 / 65536.0 - a1 / (a1 + a2)) <= 2.0 ** -16
