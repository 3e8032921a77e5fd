"""Suggest-observe loops (paper, Algorithm 1) with a synthetic objective and with the CPU checker."""
import numpy as np
import pytest

import oracle
from paper_2012_04201_b200 import driver
from paper_2012_04201_b200 import workloads as W


def synthetic(configs, sizes=None):
    """Smooth objective with its optimum inside the search space (higher is better)."""
    return -((np.log10(configs["lr"]) + 3.0) ** 2 + (np.log10(configs["alpha"]) + 2.0) ** 2
             + ((configs["hidden"] - 120.0) / 75.0) ** 2)


def test_left_algorithm_counts_and_observations():
    calls = []
    opt = driver.RandomSearch(seed=1, epochs=10)

    def ev(cfgs):
        calls.append(cfgs.size)
        return synthetic(cfgs)

    log = driver.run_study(ev, opt, n_step=16, n_batch=8)
    assert calls == [8] * 16 and len(log) == 16          # N_STEP x N_BATCH evaluations
    assert len(opt.history) == 16 and all(c.size == 8 for c, _ in opt.history)
    for cfgs, _ in log:
        assert cfgs.dtype == W.CONFIG_DTYPE and np.all(cfgs["epochs"] == 10)
        assert np.all((cfgs["hidden"] >= 50) & (cfgs["hidden"] <= 200))
        assert np.all((cfgs["beta2"] < 1.0) & (cfgs["eps"] > 0))


def test_right_algorithm_shares_observations_and_splits_the_batch():
    a = driver.RandomSearch(seed=2, epochs=5)
    b = driver.LocalPerturbation(seed=3, epochs=5)
    seen = []
    orig = b.observe
    b.observe = lambda cfgs, s: (seen.append(cfgs.size), orig(cfgs, s))
    log = driver.run_study(synthetic, [a, b], n_step=6, n_batch=8)
    assert all(c.size == 8 for c, _ in log)
    assert seen == [8] * 6                                # the second optimizer sees all 8, not its 4
    assert all(c.size == 8 for c, _ in a.history)
    with pytest.raises(ValueError):
        driver.run_study(synthetic, [a, b], n_step=1, n_batch=7)


def test_local_search_beats_random_on_a_smooth_objective():
    wins = 0
    for seed in range(8):
        r = driver.best_so_far(driver.run_study(synthetic, driver.RandomSearch(seed, 1)))[-1]
        l = driver.best_so_far(driver.run_study(synthetic, driver.LocalPerturbation(seed, 1)))[-1]
        wins += l >= r
    assert wins >= 5


def test_lockstep_studies_use_one_evaluation_per_iteration_and_match_separate_runs():
    calls = []

    def ev(cfgs, sizes):
        calls.append(list(sizes))
        return synthetic(cfgs)

    studies = [driver.LocalPerturbation(seed=s, epochs=3) for s in range(5)] + \
              [[driver.RandomSearch(50, 3), driver.LocalPerturbation(51, 3)]]
    logs = driver.run_studies(ev, studies, n_step=4, n_batch=8)
    assert calls == [[8] * 6] * 4                         # one call per iteration, 48 configurations
    alone = driver.run_study(synthetic, driver.LocalPerturbation(seed=2, epochs=3), n_step=4, n_batch=8)
    for (c1, s1), (c2, s2) in zip(logs[2], alone):
        assert np.array_equal(c1, c2) and np.array_equal(s1, s2)


def test_study_on_the_cpu_checker_improves_the_cv_score():
    wl = W.workload("iris8")

    def ev(cfgs):
        return oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], cfgs, wl["seed"])["scores"]

    log = driver.run_study(ev, [driver.RandomSearch(0, 15), driver.LocalPerturbation(1, 15)], n_step=4, n_batch=8)
    best = driver.best_so_far(log)
    assert best == sorted(best) and best[-1] >= 0.9
