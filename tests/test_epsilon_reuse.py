"""Re-use of the random samples across iterations (App. "Pruning Overhead", Part 1): what re-using a seed changes and
what it leaves alone, on the oracle.  The full study is oracle/epsilon_reuse_study.py (run it to print its table);
these tests assert its two statements on a short run."""
import numpy as np

from oracle import epsilon_reuse_study as study


def test_reuse_correlates_consecutive_errors_but_training_still_converges():
    dense = study.run(None, iters=100, run_seed=1)[0][-1]
    fresh_loss, fresh_cos = study.run(1, iters=100, run_seed=1)
    fresh_loss = fresh_loss[-1]
    reuse_loss, reuse_cos = study.run(50, iters=100, run_seed=1)
    reuse_loss = reuse_loss[-1]
    # a new eps every iteration: consecutive pruning errors are uncorrelated; a re-used eps: strongly correlated
    # (the gradient moves slowly, so the same draws keep the same elements)
    assert abs(fresh_cos) < 0.1 and reuse_cos > 0.4
    # the paper's observation: convergence is not hurt much -- both end within 15 % of dense SGD's loss, far below the start
    start = study.run(None, iters=1, run_seed=1)[0][0]
    assert dense < fresh_loss < 1.15 * dense and dense < reuse_loss < 1.15 * dense
    assert reuse_loss < 0.05 * start


def test_unbiasedness_is_over_fresh_draws():
    # the mean of n prunes of one gradient closes in on it as 1 / sqrt(n) with fresh seeds and not at all with one seed
    e1, e16 = study.averaging_on_a_fixed_gradient(1, True), study.averaging_on_a_fixed_gradient(16, True)
    assert 3.0 < e1 / e16 < 5.0
    assert study.averaging_on_a_fixed_gradient(16, False) == study.averaging_on_a_fixed_gradient(1, False) == e1
