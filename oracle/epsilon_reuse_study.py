"""Re-use of the random samples across iterations (App. "Pruning Overhead", Part 1: a new eps only every 50
iterations costs nothing in accuracy and amortises the sampling).

TEST INFRASTRUCTURE ONLY (runs the CPU oracle).  A small least-squares layer trained by SGD with its neural gradient
MVUE 2:4-pruned along the tokens before the update product; the seed of the prune changes every `refresh` iterations.
Reports, per refresh period: the final loss (mean over runs) next to dense SGD, and the correlation between the pruning
errors of consecutive iterations -- what re-use changes is that correlation, not the mean of the estimate.

    python -m oracle.epsilon_reuse_study            # prints the table
"""
from __future__ import annotations

import numpy as np

import oracle


def run(refresh: int | None, iters: int = 200, run_seed: int = 0, T: int = 256, n_in: int = 32, n_out: int = 16,
        lr: float = 0.3, joint: int = oracle.JOINT_SYSTEMATIC):
    """refresh: iterations per seed (1 = a new eps every iteration, None = dense SGD, 0 = one eps for the whole run).
    Returns (loss per iteration, mean cosine between consecutive pruning errors)."""
    rng = np.random.Generator(np.random.PCG64(1000 + run_seed))
    W_true = rng.standard_normal((n_out, n_in)).astype(np.float32)
    h = rng.standard_normal((T, n_in)).astype(np.float32)
    y = h @ W_true.T + 0.1 * rng.standard_normal((T, n_out)).astype(np.float32)
    W = np.zeros((n_out, n_in), dtype=np.float32)
    losses, cosines, prev_err = [], [], None
    for it in range(iters):
        g = ((h @ W.T - y) / T).astype(np.float32)                      # neural gradient [T x n_out]
        losses.append(float(0.5 * T * np.sum(g.astype(np.float64) ** 2)))
        if refresh is None:
            g_hat = g
        else:
            seed = 7919 * run_seed + (0 if refresh == 0 else it // refresh)
            v, m = oracle.prune(g, 2, 4, axis=0, seed=seed, joint=joint)
            g_hat = oracle.unpack(v, m).T                               # A = g^T  ->  back to [T x n_out]
            err = (g_hat - g).ravel().astype(np.float64)
            if prev_err is not None:
                cosines.append(float(err @ prev_err / (np.linalg.norm(err) * np.linalg.norm(prev_err) + 1e-300)))
            prev_err = err
        W = W - lr * (g_hat.T @ h).astype(np.float32)
    return np.array(losses), (float(np.mean(cosines)) if cosines else 0.0)


def averaging_on_a_fixed_gradient(n: int = 64, fresh: bool = True, T: int = 256, n_out: int = 16):
    """Relative error of the mean of n pruned copies of ONE gradient: falls as 1/sqrt(n) with fresh seeds, does not fall
    at all when the seed is re-used (the n copies are the same draw)."""
    g = np.random.Generator(np.random.PCG64(5)).standard_normal((T, n_out)).astype(np.float32)
    acc = np.zeros((n_out, T))
    for i in range(n):
        v, m = oracle.prune(g, 2, 4, axis=0, seed=(i if fresh else 0), joint=oracle.JOINT_SYSTEMATIC)
        acc += oracle.unpack(v, m)
    return float(np.linalg.norm(acc / n - g.T) / np.linalg.norm(g))


def table(runs: int = 5, iters: int = 200):
    rows = []
    for name, refresh in (("dense", None), ("new eps every iteration", 1), ("every 10", 10), ("every 50", 50),
                          ("one eps for the whole run", 0)):
        res = [run(refresh, iters=iters, run_seed=s) for s in range(runs)]
        rows.append((name, float(np.mean([r[0][-1] for r in res])), float(np.mean([r[1] for r in res]))))
    return rows


if __name__ == "__main__":
    print(f"{'seed refresh':28s} {'final loss':>12s} {'corr. of consecutive errors':>28s}")
    for name, loss, cos in table():
        print(f"{name:28s} {loss:12.5f} {cos:28.3f}")
    for n in (1, 4, 16, 64):
        print(f"mean of {n:2d} prunes of one gradient: rel. error fresh {averaging_on_a_fixed_gradient(n, True):.4f}  "
              f"re-used {averaging_on_a_fixed_gradient(n, False):.4f}")
