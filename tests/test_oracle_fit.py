"""Pins for whole fits in the checker: scoring, limits with known answers, invariants."""
import numpy as np

import oracle
from paper_2012_04201_b200 import workloads as W


def unpack(theta, d, H, C):
    o = 0
    W1 = theta[o:o + d * H].reshape(d, H); o += d * H
    b1 = theta[o:o + H]; o += H
    W2 = theta[o:o + H * C].reshape(H, C); o += H * C
    return W1, b1, W2, theta[o:o + C]


def one_config(hidden=8, batch_size=16, epochs=3, alpha=1e-4, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8):
    c = np.zeros(1, W.CONFIG_DTYPE)
    c[0] = (hidden, batch_size, epochs, alpha, lr, beta1, beta2, eps)
    return c


def test_scores_recomputed_by_brute_force():
    wl = W.workload("iris8")
    X, y = wl["X"], wl["y"]
    cfg = wl["configs"].copy(); cfg["epochs"] = 7
    _, fo = oracle.fold_split(150, 5, 0)
    for (c, f) in [(1, 0), (3, 4)]:
        r = oracle.cv_fits(X, y, 0, 5, cfg, 0, [c], [f], want_theta=True)
        W1, b1, W2, b2 = unpack(r["theta"], 4, int(cfg["hidden"][c]), 3)
        V = np.nonzero(fo == f)[0]
        z = np.maximum(X[V].astype(np.float64) @ W1 + b1, 0) @ W2 + b2
        acc = np.mean(np.argmax(z, 1) == y[V])
        assert abs(r["scores"][0] - acc) < 1e-6
        assert abs(r["scores"][0] * len(V) - round(r["scores"][0] * len(V))) < 1e-4
    wl = W.workload("diabetes4096", n_configs=4)
    X, y = wl["X"], wl["y"]
    cfg = wl["configs"].copy(); cfg["epochs"] = 5
    _, fo = oracle.fold_split(442, 5, 0)
    r = oracle.cv_fits(X, y, 1, 5, cfg, 0, [2], [1], mode=1, want_theta=True)
    W1, b1, W2, b2 = unpack(r["theta"], 10, int(cfg["hidden"][2]), 1)
    V = np.nonzero(fo == 1)[0]
    z = np.maximum(X[V].astype(np.float64) @ W1 + b1, 0) @ W2 + b2
    assert abs(r["scores"][0] + np.mean((z[:, 0] - y[V]) ** 2)) < 1e-12


def test_epochs_zero_scores_initial_weights_and_batch_is_clipped():
    wl = W.workload("iris8")
    X, y = wl["X"], wl["y"]
    cfg = one_config(hidden=5, epochs=0)
    r = oracle.cv_fits(X, y, 0, 5, cfg, 3, [0], [2], want_theta=True)
    assert np.array_equal(r["theta"], oracle.init_params(4, 5, 3, 3, 0, 2))
    # batch_size above the train-fold size behaves as full batch
    a = oracle.cv_fits(X, y, 0, 5, one_config(batch_size=120, epochs=4), 0, [0], [0], trace_steps=6)
    b = oracle.cv_fits(X, y, 0, 5, one_config(batch_size=150, epochs=4), 0, [0], [0], trace_steps=6)
    assert np.array_equal(a["trace"][:, :4], b["trace"][:, :4]) and a["scores"][0] == b["scores"][0]
    assert np.all(np.isnan(a["trace"][:, 4:]))  # 4 epochs x 1 step: the rest is padding


def test_step_count_and_short_last_batch():
    wl = W.workload("iris8")
    # n_train = 120, B = 50 -> 3 steps per epoch (50, 50, 20)
    r = oracle.cv_fits(wl["X"], wl["y"], 0, 5, one_config(batch_size=50, epochs=2), 0, [0], [0], trace_steps=8)
    assert np.isfinite(r["trace"][0, :6]).all() and np.isnan(r["trace"][0, 6:]).all()


def test_minibatch_fit_replayed_step_by_step():
    # A fit with several minibatches per epoch and a short last batch (120 training rows, B = 50:
    # 50, 50, 20), replayed outside the fit loop from its parts: the epoch order export, the
    # minibatch loss/gradient export and the Adam export (double mode, so that the comparison is
    # not about rounding).  Pins the slicing rows = order[s B : (s+1) B], the per-batch mean over
    # the true batch size, the step counter running across epochs and the reshuffle per epoch.
    wl = W.workload("iris8")
    X, y = wl["X"].astype(np.float64), wl["y"].astype(np.float64)
    cfg = one_config(hidden=6, batch_size=50, epochs=2, alpha=0.3, lr=0.02, beta1=0.8, beta2=0.95, eps=1e-7)
    config, fold, seed = 0, 3, 11
    r = oracle.cv_fits(wl["X"], wl["y"], 0, 5, cfg, seed, [config], [fold], mode=1, trace_steps=8, want_theta=True)
    th0 = oracle.init_params(4, 6, 3, seed, config, fold)
    hp = [float(np.float32(v)) for v in (0.02, 0.8, 0.95, 1e-7)]
    grads, losses = [], []
    for e in range(2):
        order = oracle.epoch_order(150, 5, seed, config, fold, e)
        assert len(order) == 120
        for s in range(3):
            rows = order[s * 50:(s + 1) * 50]
            assert len(rows) == (50, 50, 20)[s]
            th = th0 if not grads else oracle.adam_steps(1, th0, np.zeros_like(th0), np.zeros_like(th0), np.array(grads), *hp)[0]
            loss, g = oracle.loss_grad(1, 4, 6, 3, 0, float(np.float32(0.3)), th, X[rows], y[rows])
            grads.append(g); losses.append(loss)
    th_final = oracle.adam_steps(1, th0, np.zeros_like(th0), np.zeros_like(th0), np.array(grads), *hp)[0]
    np.testing.assert_allclose(r["trace"][0, :6], losses, rtol=1e-12)
    assert np.all(np.isnan(r["trace"][0, 6:]))
    np.testing.assert_allclose(r["theta"], th_final, rtol=1e-11, atol=1e-13)
    # a wrong slice (e.g. dropping the short batch, or reusing epoch 0's order) would not reproduce it
    assert not np.array_equal(oracle.epoch_order(150, 5, seed, config, fold, 0), oracle.epoch_order(150, 5, seed, config, fold, 1))


def test_diverged_fits_nan_maps_to_minus_infinity_and_class_zero():
    # A learning rate of 1e20 turns the parameters into NaN within a few steps.  Regression: the
    # held-out error is NaN and the score is -inf (never NaN).  Classification: every logit is NaN,
    # NaN never wins the ascending strict-> scan, so the prediction is class 0 (the lowest index,
    # which is also what a tie between equal logits gives) and the accuracy is the share of
    # class-0 rows in the held-out fold.
    wl = W.workload("diabetes4096", n_configs=1)
    cfg = one_config(hidden=6, epochs=40, lr=1e20, batch_size=64)
    r = oracle.cv_fits(wl["X"], wl["y"], 1, 5, cfg, 0, [0, 0], [0, 1], want_theta=True)
    assert np.isnan(r["theta"]).any()
    assert np.all(np.isneginf(r["scores"]))
    ev = oracle.cv_eval(wl["X"], wl["y"], 1, 5, cfg, 0)
    assert np.isneginf(ev["scores"][0]) and not np.isnan(ev["fold_scores"]).any()
    wl = W.workload("iris8")
    _, fo = oracle.fold_split(150, 5, 0)
    r = oracle.cv_fits(wl["X"], wl["y"], 0, 5, cfg, 0, [0, 0], [0, 1], want_theta=True)
    assert np.isnan(r["theta"]).any()
    for f, score in zip((0, 1), r["scores"]):
        assert abs(score - np.mean(wl["y"][fo == f] == 0)) < 1e-6


def test_float_and_double_traces_agree_over_50_steps():
    wl = W.workload("breast128", n_configs=6)
    a = oracle.cv_eval(wl["X"], wl["y"], 0, 5, wl["configs"], 0, mode=0, trace_steps=50)
    b = oracle.cv_eval(wl["X"], wl["y"], 0, 5, wl["configs"], 0, mode=1, trace_steps=50)
    ok = np.isfinite(b["trace"])
    rel = np.abs(a["trace"][ok] - b["trace"][ok]) / np.abs(b["trace"][ok])
    assert rel.max() < 1e-3 and np.median(rel) < 1e-5


def test_huge_alpha_shrinks_weights_alpha_zero_keeps_path():
    wl = W.workload("iris8")
    X, y = wl["X"], wl["y"]
    norms = []
    for e in (0, 40, 400):
        r = oracle.cv_fits(X, y, 0, 5, one_config(hidden=6, batch_size=120, epochs=e, alpha=1e4, lr=5e-3),
                           0, [0], [0], want_theta=True)
        W1, b1, W2, b2 = unpack(r["theta"], 4, 6, 3)
        norms.append(np.sqrt((W1 ** 2).sum() + (W2 ** 2).sum()))
    assert norms[0] > 1.0 and norms[1] < norms[0] and norms[2] < 0.1


def test_separable_data_drives_training_loss_to_zero():
    # two well separated blobs, full batch, alpha = 0: cross-entropy must vanish
    rng = np.random.default_rng(0)
    X = np.concatenate([rng.normal(-4, 0.5, (20, 2)), rng.normal(4, 0.5, (20, 2))]).astype(np.float32)
    y = np.repeat([0.0, 1.0], 20).astype(np.float32)
    cfg = one_config(hidden=16, batch_size=1000, epochs=400, alpha=0.0, lr=0.05)
    r = oracle.cv_fits(X, y, 0, 4, cfg, 0, [0] * 4, [0, 1, 2, 3], trace_steps=400)
    assert np.all(r["trace"][:, -1] < 1e-3) and np.all(r["scores"] == 1.0)
    assert np.all(r["trace"][:, 0] > 0.1)


def test_regression_on_linear_data_approaches_least_squares():
    rng = np.random.default_rng(1)
    n, d = 200, 3
    X = rng.normal(size=(n, d)).astype(np.float32)
    y = (X @ np.array([1.0, -2.0, 0.5]) + 0.3 + rng.normal(0, 0.1, n)).astype(np.float32)
    cfg = one_config(hidden=32, batch_size=40, epochs=300, alpha=0.0, lr=0.01)
    r = oracle.cv_eval(X, y, 1, 5, cfg, 0, mode=1)
    _, fo = oracle.fold_split(n, 5, 0)
    ls = []
    for f in range(5):
        tr, va = fo != f, fo == f
        A = np.c_[X[tr], np.ones(tr.sum())]
        w, *_ = np.linalg.lstsq(A, y[tr], rcond=None)
        ls.append(-np.mean((np.c_[X[va], np.ones(va.sum())] @ w - y[va]) ** 2))
    # the net contains the linear model; its held-out error is close to the least-squares one
    assert np.all(r["fold_scores"][0] > np.array(ls) - 0.02)
    assert np.all(r["fold_scores"][0] < 0.0) and r["scores"][0] > -0.04


def test_determinism_threads_and_config_independence():
    wl = W.workload("iris8")
    X, y, cfg = wl["X"], wl["y"], wl["configs"].copy()
    cfg["epochs"] = 5
    a = oracle.cv_eval(X, y, 0, 5, cfg, 0, n_threads=1, trace_steps=3)
    b = oracle.cv_eval(X, y, 0, 5, cfg, 0, n_threads=4, trace_steps=3)
    assert np.array_equal(a["fold_scores"], b["fold_scores"]) and np.array_equal(a["trace"], b["trace"])
    # score of config c depends on its index and content only, not on the rest of the list
    sub = cfg[:3].copy()
    sub[0] = cfg[5]
    c = oracle.cv_eval(X, y, 0, 5, sub, 0)
    assert np.array_equal(c["fold_scores"][1:3], a["fold_scores"][1:3])
    # mean over folds, float arithmetic in fold order
    m = np.float32(0)
    for f in range(5):
        m = np.float32(m + np.float32(a["fold_scores"][2, f]))
    assert a["scores"][2] == float(np.float32(m / np.float32(5)))
    # the seed matters
    assert not np.array_equal(oracle.cv_eval(X, y, 0, 5, cfg, 1)["fold_scores"], a["fold_scores"])


def test_invalid_arguments_rejected():
    wl = W.workload("iris8")
    import pytest
    bad = wl["configs"].copy(); bad["beta2"][0] = 1.0
    with pytest.raises(ValueError):
        oracle.cv_eval(wl["X"], wl["y"], 0, 5, bad, 0)
    with pytest.raises(ValueError):
        oracle.cv_eval(wl["X"], wl["y"], 0, 1, wl["configs"], 0)
    with pytest.raises(ValueError):
        oracle.cv_eval(wl["X"], wl["y"] - 0.5, 0, 5, wl["configs"], 0)
