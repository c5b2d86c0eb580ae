"""Monte Carlo over seeds on the 16x16 slice of the small linear-layer workload."""
import numpy as np
import pytest

import oracle
from oracle import theory
from paper_2203_10991_b200 import workloads

N_SEEDS = 10000


def _slice():
    cfg = workloads.CONFIGS["linear_small"]
    g = workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype="f32")
    return np.ascontiguousarray(g[:16, :16])


@pytest.mark.parametrize("n,m,joint", [(1, 2, 0), (2, 4, 0), (2, 4, 1)])
def test_mean_and_mask_frequencies_over_seeds(n, m, joint):
    g = _slice()
    acc = np.zeros((16, 16))
    nib_counts = np.zeros((16, 4, 16))                    # [A row, group, nibble value]
    for seed in range(N_SEEDS):
        values, meta = oracle.prune(g, n, m, axis=0, seed=seed, joint=joint)       # A = g^T: [16, 16]
        acc += oracle.unpack(values, meta)
        nibs = np.stack([meta & 0xF, meta >> 4], axis=2).reshape(16, 4)
        for r in range(16):
            for j in range(4):
                nib_counts[r, j, nibs[r, j]] += 1
    mean = acc / N_SEEDS
    A = g.T.astype(np.float64)
    for r in range(16):
        for j in range(4):
            blk = A[r, 4 * j:4 * j + 4]
            if m == 4:
                p = theory.marginals24(blk)
                law_of = theory.outcome_law24 if joint == oracle.JOINT_TABLE else theory.systematic_law24
                law = law_of(blk) if np.count_nonzero(blk) >= 2 else None
            else:
                p = np.zeros(4)
                for h in range(2):
                    s = abs(blk[2 * h]) + abs(blk[2 * h + 1])
                    if s > 0:
                        p[2 * h], p[2 * h + 1] = abs(blk[2 * h]) / s, abs(blk[2 * h + 1]) / s
                law = None
            for e in range(4):
                a = blk[e]
                if a == 0:
                    assert mean[r, 4 * j + e] == 0
                    continue
                sd = np.sqrt(a * a * (1 / p[e] - 1) / N_SEEDS)
                assert abs(mean[r, 4 * j + e] - a) <= 6 * sd + 2.0**-8 * abs(a)
            if law is not None:
                for (i0, i1), pr in law.items():
                    f = nib_counts[r, j, i0 | (i1 << 2)] / N_SEEDS
                    assert abs(f - pr) <= 6 * np.sqrt(max(pr * (1 - pr), 1e-12) / N_SEEDS) + 1e-9


def test_greedy_and_biased_would_fail_the_same_check():
    # power of the check above: replace the estimator by Table 2's biased ones and the bound breaks
    g = _slice()
    A = g.T.astype(np.float64)
    violations = {"greedy": 0, "biased": 0}
    for r in range(16):
        for j2 in range(8):
            a1, a2 = A[r, 2 * j2], A[r, 2 * j2 + 1]
            if a1 == 0 or a2 == 0:
                continue
            p1 = abs(a1) / (abs(a1) + abs(a2))
            for name in violations:
                mean, _ = theory.mean_and_variance(theory.estimator12(name, a1, a2))
                sd = np.sqrt(a1 * a1 * (1 / p1 - 1) / N_SEEDS)
                if abs(mean[0] - a1) > 6 * sd + 2.0**-8 * abs(a1):
                    violations[name] += 1
    assert violations["greedy"] > 5 and violations["biased"] > 5
