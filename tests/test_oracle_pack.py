"""Pins for bf16 rounding, the canonical packed form and tensor-wide block numbering."""
import numpy as np
import pytest
import torch

import oracle
from oracle import philox_py
from paper_2203_10991_b200 import workloads


def test_bf16_rne_matches_library_cast():
    rng = np.random.Generator(np.random.PCG64(3))
    bits = rng.integers(0, 2**32, 200000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    edge = np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 1.0078125, 3.3895314e38, 1e-40, -1e-45,
                     np.float32(1 + 2**-8), np.float32(1 + 2**-8 + 2**-20), np.float32(1 + 3 * 2**-8)],
                    dtype=np.float32)
    x = np.concatenate([x, edge])
    got = oracle.bf16_rne(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    # round trip of every bf16 finite pattern is the identity
    allb = np.arange(0, 1 << 16, dtype=np.uint16)
    f = oracle.bf16_to_f32(allb)
    fin = np.isfinite(f)
    assert np.array_equal(oracle.bf16_rne(f[fin]), allb[fin])


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1)])
@pytest.mark.parametrize("dist", ["relu_normal", "relu_lognormal", "student_t"])
def test_packed_form_properties(n, m, joint, dist):
    g = workloads.gradient((48, 64), dist, seed=9, dtype="bf16")
    values, meta = oracle.prune(g, n, m, axis=1, seed=5, joint=joint)
    assert values.shape == (48, 32) and meta.shape == (48, 8)
    lo, hi = meta & 3, (meta >> 2) & 3
    lo2, hi2 = (meta >> 4) & 3, (meta >> 6) & 3
    assert (lo < hi).all() and (lo2 < hi2).all()              # ascending positions inside a group
    if m == 2:                                                # 1:2 written as a valid 2:4 pattern
        assert (lo <= 1).all() and (hi >= 2).all() and (lo2 <= 1).all() and (hi2 >= 2).all()
    dense = oracle.unpack(values, meta)
    assert dense.shape == (48, 64)
    gf = oracle.bf16_to_f32(g)
    grp = dense.reshape(48, 16, 4)
    assert (np.count_nonzero(grp, axis=2) <= 2).all()
    # a survivor keeps the sign of its source and never has a smaller magnitude
    nz = dense != 0
    assert (np.sign(dense[nz]) == np.sign(gf[nz])).all()
    assert (np.abs(dense[nz]) >= np.abs(gf[nz]) * (1 - 2.0**-8)).all()
    # a zero source is never turned into a non-zero
    assert (dense[gf == 0] == 0).all()
    # per group: the sum of magnitudes is preserved up to bf16 rounding when >= 2 non-zeros exist (uncapped
    # groups keep two copies of sum/2; capped groups keep max + rest)
    src = np.abs(gf).reshape(48, 16, 4)
    if m == 4:
        tot_src = src.sum(2)
        tot_out = np.abs(grp).sum(2)
        assert np.allclose(tot_out, tot_src, rtol=2.0**-7, atol=0)


def test_prune_agrees_with_per_block_calls_and_numbering():
    # tensor-wide loop == block sampler driven by word(seed, q), q = r * (K/M) + j
    g = workloads.gradient((8, 32), "student_t", seed=4, dtype="f32")
    seed = 0xDEADBEEFCAFE
    for joint in (oracle.JOINT_TABLE, oracle.JOINT_SYSTEMATIC):
        values, meta = oracle.prune(g, 2, 4, axis=1, seed=seed, joint=joint)
        for r in range(8):
            for j in range(8):
                q = r * 8 + j
                (i0, i1), (v0, v1) = oracle.mvue_2of4(g[r, 4 * j:4 * j + 4], philox_py.block_word(seed, q), joint)
                nib = (meta[r, j // 2] >> (4 * (j % 2))) & 0xF
                assert nib == (i0 | (i1 << 2))
                assert values[r, 2 * j] == oracle.bf16_rne(np.float32(v0))
                assert values[r, 2 * j + 1] == oracle.bf16_rne(np.float32(v1))
    values, meta = oracle.prune(g, 1, 2, axis=1, seed=seed)
    for r in range(8):
        for j2 in range(16):
            q = r * 16 + j2
            idx, kept = oracle.mvue_1of2(g[r, 2 * j2], g[r, 2 * j2 + 1], philox_py.block_word(seed, q))
            j = j2 // 2
            nib = (meta[r, j // 2] >> (4 * (j % 2))) & 0xF
            two_bit = (nib >> (2 * (j2 % 2))) & 3
            assert two_bit == 2 * (j2 % 2) + idx
            assert values[r, j2] == oracle.bf16_rne(np.float32(kept))


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1)])
def test_axis0_is_the_transpose_view(n, m, joint):
    # blocks down the rows of g == blocks along the rows of g^T, same block numbers
    g = workloads.gradient((64, 24), "relu_normal", seed=1, dtype="bf16")
    v0, m0 = oracle.prune(g, n, m, axis=0, seed=3, joint=joint)
    v1, m1 = oracle.prune(np.ascontiguousarray(g.T), n, m, axis=1, seed=3, joint=joint)
    assert np.array_equal(v0, v1) and np.array_equal(m0, m1)
    assert v0.shape == (24, 32) and m0.shape == (24, 8)


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1)])
def test_k_shards_reproduce_the_unsharded_masks(n, m, joint):
    g = workloads.gradient((96, 16), "student_t", seed=2, dtype="bf16")
    v, mt = oracle.prune(g, n, m, axis=0, seed=8, joint=joint)
    for lo, hi in [(0, 32), (32, 96)]:
        vs, ms = oracle.prune(g[lo:hi], n, m, axis=0, seed=8, k_total=96, k_offset=lo, joint=joint)
        assert np.array_equal(vs, v[:, lo // 2:hi // 2]) and np.array_equal(ms, mt[:, lo // 8:hi // 8])


def test_threads_do_not_change_the_result_and_seed_does():
    g = workloads.gradient((64, 64), "student_t", seed=2, dtype="bf16")
    a = oracle.prune(g, 2, 4, axis=1, seed=1, threads=1)
    b = oracle.prune(g, 2, 4, axis=1, seed=1, threads=4)
    c = oracle.prune(g, 2, 4, axis=1, seed=2, threads=1)
    d = oracle.prune(g, 2, 4, axis=1, seed=1, threads=1, joint=oracle.JOINT_SYSTEMATIC)
    e = oracle.prune(g, 1, 2, axis=1, seed=1), oracle.prune(g, 1, 2, axis=1, seed=1, joint=oracle.JOINT_SYSTEMATIC)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(a[1], c[1])
    assert not np.array_equal(a[1], d[1])                      # the two 2:4 laws draw different pairs
    assert np.array_equal(e[0][0], e[1][0]) and np.array_equal(e[0][1], e[1][1])   # 1:2 has one law


def test_unsupported_modes_are_rejected():
    g = np.zeros((16, 16), dtype=np.float32)
    for n, m in [(3, 4), (4, 8), (2, 2), (0, 4)]:
        with pytest.raises(ValueError):
            oracle.prune(g, n, m, axis=1, seed=0)
    with pytest.raises(ValueError):
        oracle.prune(np.zeros((16, 12), dtype=np.float32), 2, 4, axis=1, seed=0)
