"""CUDA path against the CPU checker for the variants of the evaluation: the SGD solver
(paper Table 1: MLP-sgd) and the nll / mae held-out metrics (paper Table 1), through the C ABI.

Same bars as the main parity tests: training loss of the first 50 steps within 1e-4 relative,
fold scores within 1e-3 absolute for at least 99 % of fits.  The SGD update and the absolute
error are fixed-order float arithmetic on both sides (bit-equality is reported); the
log-likelihood goes through each side's own logarithm, so only the tolerance applies to it.
"""
import numpy as np
import pytest

import oracle
from paper_2012_04201_b200 import workloads as W
from test_gpu_parity import check_against_oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2012_04201_b200 import binding as b
    return b


def gpu_eval(binding, wl, configs, trace_steps=0, keep_theta=False, solver=0, metric=0):
    h = binding.MlpCv(trace_steps=trace_steps, keep_theta=keep_theta, solver=solver, metric=metric)
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    scores = h.eval(X, y, wl["task"], wl["n_folds"], configs, wl["seed"]).cpu().numpy()
    out = dict(scores=scores, fold_scores=h.fold_scores())
    if trace_steps:
        out["trace"] = h.loss_trace()
    if keep_theta:
        C = 1 if wl["task"] == 1 else int(wl["y"].max()) + 1
        out["theta"] = h.debug_theta(oracle.param_count(wl["X"].shape[1], int(configs[-1]["hidden"]), C))
    h.close()
    return out


def sgd_configs(wl, n, epochs):
    cfg = wl["configs"][:n].copy()
    cfg["epochs"] = epochs
    cfg["lr"] = np.minimum(cfg["lr"], 0.02)  # plain SGD diverges at the upper end of Adam's range
    return cfg


@pytest.mark.parametrize("name,n_cfg,epochs", [("iris8", 8, 30), ("breast128", 16, 12), ("diabetes4096", 24, 10),
                                               ("digits2048", 6, 3)])
def test_sgd_solver_matches_checker(binding, name, n_cfg, epochs):
    wl = W.workload(name, n_configs=max(n_cfg, 8)) if name != "iris8" else W.workload(name)
    cfg = sgd_configs(wl, n_cfg, epochs)
    gpu = gpu_eval(binding, wl, cfg, trace_steps=50, keep_theta=True, solver=binding.SOLVER_SGD)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], cfg, wl["seed"], trace_steps=50,
                         solver=oracle.SOLVER_SGD)
    check_against_oracle(gpu, ref, name + "/sgd")
    K = wl["n_folds"]
    th = oracle.cv_fits(wl["X"], wl["y"], wl["task"], K, cfg, wl["seed"], [n_cfg - 1], [K - 1], want_theta=True,
                        solver=oracle.SOLVER_SGD)["theta"]
    print(f"[{name}/sgd] final parameters bit-equal:", np.array_equal(gpu["theta"].astype(np.float64), th))
    fin = np.isfinite(th)
    np.testing.assert_allclose(gpu["theta"][fin], th[fin], rtol=1e-3, atol=1e-4)
    # the solver option changes the result (the Adam path was not taken by mistake)
    adam = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], cfg, wl["seed"])
    assert not np.array_equal(adam["fold_scores"], ref["fold_scores"])


@pytest.mark.parametrize("name,n_cfg,epochs,solver", [("iris8", 8, 25, 0), ("digits2048", 6, 3, 0),
                                                      ("diabetes4096", 24, 10, 0), ("breast128", 12, 8, 1)])
def test_nll_and_mae_metrics_match_checker(binding, name, n_cfg, epochs, solver):
    wl = W.workload(name, n_configs=max(n_cfg, 8)) if name != "iris8" else W.workload(name)
    cfg = sgd_configs(wl, n_cfg, epochs) if solver else wl["configs"][:n_cfg].copy()
    cfg["epochs"] = epochs
    gpu = gpu_eval(binding, wl, cfg, solver=solver, metric=binding.METRIC_ALT)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], cfg, wl["seed"], solver=solver,
                         metric=oracle.METRIC_ALT)
    check_against_oracle(gpu, ref, name + "/alt-metric")
    assert np.all(gpu["fold_scores"][np.isfinite(gpu["fold_scores"])] <= 0.0)
    # same training as with the default metric: the scores differ, and for regression the two
    # errors of one fit obey mean|r| <= sqrt(mean r^2)
    base = gpu_eval(binding, wl, cfg, solver=solver)
    if wl["task"] == 1:
        mae, mse = -gpu["fold_scores"].astype(np.float64), -base["fold_scores"].astype(np.float64)
        fin = np.isfinite(mae) & np.isfinite(mse)
        assert np.all(mae[fin] <= np.sqrt(mse[fin]) * (1 + 1e-5))
    else:
        assert not np.array_equal(gpu["fold_scores"], base["fold_scores"])


@pytest.mark.parametrize("name", ["housing10k", "collider10k"])
def test_ten_thousand_row_shape_matches_checker(binding, name):
    # the shape of the paper's down-sampled 10,000-row sets: 8,000-row training folds, so the
    # per-epoch permutation sorts 8,000 keys and a fit takes up to 800 steps per epoch
    wl = W.workload(name, n_configs=12, epochs=3)
    cfg = wl["configs"]
    h = binding.MlpCv()
    for config, fold, epoch in [(0, 0, 0), (11, 4, 2)]:
        fo, order = h.debug_indices(10000, 5, wl["seed"], config, fold, epoch)
        assert np.array_equal(fo, oracle.fold_split(10000, 5, wl["seed"])[1])
        assert np.array_equal(order, oracle.epoch_order(10000, 5, wl["seed"], config, fold, epoch))
    h.close()
    gpu = gpu_eval(binding, wl, cfg, trace_steps=50, keep_theta=True)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, cfg, wl["seed"], trace_steps=50)
    exact = check_against_oracle(gpu, ref, name)
    th = oracle.cv_fits(wl["X"], wl["y"], wl["task"], 5, cfg, wl["seed"], [11], [4], want_theta=True)["theta"]
    print(f"[{name}] fold scores bit-equal {exact:.3f}; final parameters bit-equal:",
          np.array_equal(gpu["theta"].astype(np.float64), th))
    np.testing.assert_allclose(gpu["theta"], th, rtol=1e-3, atol=1e-4)


@pytest.mark.parametrize("name,n_train,metric,solver", [("iris8", 110, 0, 0), ("digits2048", 1500, 1, 0),
                                                        ("diabetes4096", 401, 0, 0), ("breast128", 450, 0, 1),
                                                        ("diabetes4096", 390, 1, 0)])
def test_holdout_scores_match_checker(binding, name, n_train, metric, solver):
    # paper sec. 6.2: train on the optimisation part, score the held-out part
    wl = W.workload(name, n_configs=10) if name != "iris8" else W.workload(name)
    X, y = wl["X"], wl["y"]
    cfg = sgd_configs(wl, 8, 6) if solver else wl["configs"][:8].copy()
    cfg["epochs"] = 6 if name != "digits2048" else 2
    h = binding.MlpCv(keep_theta=True, solver=solver, metric=metric)
    Xd, yd = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    got = h.eval_holdout(Xd[:n_train], yd[:n_train], Xd[n_train:], yd[n_train:], wl["task"], cfg, wl["seed"]).cpu().numpy()
    C = 1 if wl["task"] == 1 else int(y.max()) + 1
    theta = h.debug_theta(oracle.param_count(X.shape[1], int(cfg[-1]["hidden"]), C))
    per_fit = h.fold_scores()
    h.close()
    ref = oracle.holdout_eval(X[:n_train], y[:n_train], X[n_train:], y[n_train:], wl["task"], cfg, wl["seed"],
                              solver=solver, metric=metric, want_theta=True)
    assert np.array_equal(per_fit.ravel(), got)
    both_inf = np.isinf(got) & np.isinf(ref["scores"])
    err = np.where(both_inf, 0.0, np.abs(got.astype(np.float64) - ref["scores"]))
    print(f"[{name}/holdout] max err {err.max():.3g}, bit-equal {np.mean((got.astype(np.float64) == ref['scores']) | both_inf):.3f};"
          f" parameters bit-equal: {np.array_equal(theta.astype(np.float64), ref['theta'])}")
    assert np.mean(err <= 1e-3) >= 0.99
    fin = np.isfinite(ref["theta"])
    np.testing.assert_allclose(theta[fin], ref["theta"][fin], rtol=1e-3, atol=1e-4)


def test_option_values_are_validated(binding):
    with pytest.raises(binding.BboError):
        binding.MlpCv(solver=2)
    with pytest.raises(binding.BboError):
        binding.MlpCv(metric=-1)
