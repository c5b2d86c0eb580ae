"""Pins for the oracle's product (Sec. 1: update g h^T and backward W^T g)."""
import numpy as np

import oracle
from paper_2203_10991_b200 import workloads


def test_matches_library_fp64_matmul():
    g = workloads.gradient((64, 40), "student_t", seed=1, dtype="bf16")      # [T, out]
    h = workloads.normal_bf16((64, 24), seed=2)                              # [T, in]
    values, meta = oracle.prune(g, 2, 4, axis=0, seed=3)                     # A = theta(g)^T [out, T]
    A = oracle.unpack(values, meta)
    C = oracle.gemm(A, h)
    want = A.astype(np.float64) @ oracle.bf16_to_f32(h).astype(np.float64)
    assert C.shape == (40, 24)
    assert np.allclose(C, want, rtol=1e-12, atol=1e-15)
    E = workloads.normal_bf16((40, 24), seed=5)
    C2 = oracle.gemm(A, h, E)
    assert np.allclose(C2, want * oracle.bf16_to_f32(E), rtol=1e-12, atol=1e-15)
    assert abs(oracle.gemm_entry(A[7], h, 11) - want[7, 11]) <= 1e-12 * abs(want[7, 11]) + 1e-18
    assert np.array_equal(oracle.gemm(A, h, threads=3), C)


def test_one_hot_probes_fix_operand_orientation():
    # A single non-zero in A and in B pins which index is which (a transposed operand fails)
    M, K, N = 5, 8, 7
    for (i, k, j) in [(0, 0, 0), (4, 7, 6), (2, 5, 1), (3, 1, 4)]:
        A = np.zeros((M, K), dtype=np.float32)
        B = np.zeros((K, N), dtype=np.float32)
        A[i, k] = 2.0
        B[k, j] = 3.0
        C = oracle.gemm(A, workloads.to_bf16_bits(B))
        want = np.zeros((M, N))
        want[i, j] = 6.0
        assert np.array_equal(C, want)


def test_pruned_update_is_unbiased_over_seeds():
    # E[theta(g)^T h] = g^T h (Sec. 3: an unbiased neural gradient gives an unbiased weight gradient)
    g = workloads.gradient((32, 8), "relu_normal", seed=6, dtype="bf16")
    h = workloads.normal_bf16((32, 8), seed=7)
    exact = oracle.bf16_to_f32(g).astype(np.float64).T @ oracle.bf16_to_f32(h).astype(np.float64)
    acc = np.zeros_like(exact)
    acc2 = np.zeros_like(exact)
    n = 3000
    for seed in range(n):
        values, meta = oracle.prune(g, 2, 4, axis=0, seed=seed)
        C = oracle.gemm(oracle.unpack(values, meta), h)
        acc += C
        acc2 += C * C
    mean = acc / n
    sd = np.sqrt(np.maximum(acc2 / n - mean**2, 0) / n)
    # 6 sigma plus the bf16 storage error of the survivors (relative 2^-9 per term)
    bound = 6 * sd + 2.0**-8 * (np.abs(oracle.bf16_to_f32(g)).astype(np.float64).T
                                 @ np.abs(oracle.bf16_to_f32(h)).astype(np.float64))
    assert (np.abs(mean - exact) <= bound).all()
