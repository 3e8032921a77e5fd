"""Seeded synthetic inputs: datasets and hyperparameter suggestions.

This module holds input generators only -- none of the method's arithmetic --
so that both the CUDA path and the CPU checker can be fed identical arrays.
Everything is drawn from ``numpy.random.default_rng(seed)``.

The datasets are stand-ins with the shape, size, class balance and value
range of the small tabular sets the paper evaluates on (Table 1: iris-,
breast-, digits- and diabetes-shaped); no record of those sets is reproduced.
The hyperparameter sampler plays the role of ``opt.suggest(n)`` in
Algorithm 1: it returns a ``params_list`` as a structured array.
"""
from __future__ import annotations

import numpy as np

TASK_CLASSIFICATION = 0
TASK_REGRESSION = 1

#: POD layout of one suggested configuration (32 bytes, little endian).
CONFIG_DTYPE = np.dtype(
    [
        ("hidden", "<i4"),
        ("batch_size", "<i4"),
        ("epochs", "<i4"),
        ("alpha", "<f4"),
        ("lr", "<f4"),
        ("beta1", "<f4"),
        ("beta2", "<f4"),
        ("eps", "<f4"),
    ],
    align=False,
)
assert CONFIG_DTYPE.itemsize == 32


def suggest_configs(n_configs, seed, epochs, batch_hi=150, hidden=None, batch_size=None):
    """Draw ``n_configs`` hyperparameter suggestions.

    Ranges: hidden U{50..200}; alpha log-U[1e-5, 1e1]; batch_size U{10..batch_hi};
    lr log-U[1e-5, 1e-1]; beta1 U[0.5, 0.99]; beta2 U[0.9, 0.999999];
    eps log-U[1e-9, 1e-6].  ``hidden`` / ``batch_size`` pin that field to a
    constant (throughput sweeps).  All columns are drawn even when pinned so
    the other fields do not depend on the pinning.
    """
    rng = np.random.default_rng(seed)
    out = np.zeros(n_configs, dtype=CONFIG_DTYPE)
    h = rng.integers(50, 201, size=n_configs)
    alpha = 10.0 ** rng.uniform(-5.0, 1.0, size=n_configs)
    b = rng.integers(10, batch_hi + 1, size=n_configs)
    lr = 10.0 ** rng.uniform(-5.0, -1.0, size=n_configs)
    beta1 = rng.uniform(0.5, 0.99, size=n_configs)
    beta2 = rng.uniform(0.9, 0.999999, size=n_configs)
    eps = 10.0 ** rng.uniform(-9.0, -6.0, size=n_configs)
    out["hidden"] = h if hidden is None else hidden
    out["batch_size"] = b if batch_size is None else batch_size
    out["epochs"] = epochs
    out["alpha"] = alpha.astype(np.float32)
    out["lr"] = lr.astype(np.float32)
    out["beta1"] = beta1.astype(np.float32)
    # float32 rounding may push beta2 to exactly 1.0; keep it strictly below.
    out["beta2"] = np.minimum(beta2.astype(np.float32), np.float32(0.99999994))
    out["eps"] = eps.astype(np.float32)
    return out


def blobs_iris_shaped(seed=0):
    """150 x 4, three balanced classes: isotropic unit-variance Gaussian blobs
    around class means ~ N(0, 3^2 I)."""
    rng = np.random.default_rng(seed)
    n_per, d, n_cls = 50, 4, 3
    means = rng.normal(0.0, 3.0, size=(n_cls, d))
    X = np.concatenate([means[c] + rng.normal(size=(n_per, d)) for c in range(n_cls)])
    y = np.repeat(np.arange(n_cls), n_per)
    p = rng.permutation(X.shape[0])
    return X[p].astype(np.float32), y[p].astype(np.float32)


def gaussians_breast_shaped(seed=0):
    """569 x 30, two classes (211 / 358): correlated Gaussians with a random
    covariance Q diag(lam) Q^T (Q from a QR factorisation, lam ~ U[0.5, 2]),
    class means 1.5 sigma apart along a random direction, then standardised
    per feature."""
    rng = np.random.default_rng(seed)
    d, counts = 30, (211, 358)
    parts, labels = [], []
    direction = rng.normal(size=d)
    direction /= np.linalg.norm(direction)
    for c, m in enumerate(counts):
        q, _ = np.linalg.qr(rng.normal(size=(d, d)))
        lam = rng.uniform(0.5, 2.0, size=d)
        z = rng.normal(size=(m, d)) * np.sqrt(lam)
        sigma_dir = np.sqrt(direction @ (q * lam) @ q.T @ direction)
        parts.append(z @ q.T + (c - 0.5) * 1.5 * sigma_dir * direction)
        labels.append(np.full(m, c))
    X = np.concatenate(parts)
    y = np.concatenate(labels)
    X = (X - X.mean(0)) / X.std(0)
    p = rng.permutation(X.shape[0])
    return X[p].astype(np.float32), y[p].astype(np.float32)


def digits_shaped(seed=0):
    """1797 x 64, ten classes (180 x 7 + 179 x 3): integer intensities 0..16
    (per-class Poisson-like 8x8 prototype with a dark border, plus N(0, 2^2)
    noise, rounded and clipped), scaled to [0, 1]."""
    rng = np.random.default_rng(seed)
    counts = [180] * 7 + [179] * 3
    border = np.ones((8, 8))
    border[:, 0] = border[:, 7] = 0.15
    border[0, :] *= 0.6
    border[7, :] *= 0.6
    parts, labels = [], []
    for c, m in enumerate(counts):
        proto = np.minimum(rng.poisson(6.0, size=(8, 8)) * border * 1.4, 16.0).reshape(64)
        sample = np.clip(np.rint(proto + rng.normal(0.0, 2.0, size=(m, 64))), 0, 16)
        parts.append(sample / 16.0)
        labels.append(np.full(m, c))
    X = np.concatenate(parts)
    y = np.concatenate(labels)
    p = rng.permutation(X.shape[0])
    return X[p].astype(np.float32), y[p].astype(np.float32)


def linear_diabetes_shaped(seed=0):
    """442 x 10 regression: standardised Gaussian features, y = X w + N(0, 0.5^2)
    with w ~ N(0, I), y standardised."""
    rng = np.random.default_rng(seed)
    n, d = 442, 10
    X = rng.normal(size=(n, d))
    X = (X - X.mean(0)) / X.std(0)
    w = rng.normal(size=d)
    y = X @ w + rng.normal(0.0, 0.5, size=n)
    y = (y - y.mean()) / y.std()
    return X.astype(np.float32), y.astype(np.float32)


def housing_shaped(seed=0):
    """10,000 x 8 regression (the shape of the paper's down-sampled 10,000-row sets): standardised
    features, half of them log-normal before standardisation (skewed, as counts and incomes
    are), target = a smooth non-linear function of three features plus N(0, 0.3^2),
    standardised."""
    rng = np.random.default_rng(seed)
    n, d = 10000, 8
    X = rng.normal(size=(n, d))
    X[:, :4] = np.exp(0.5 * X[:, :4])
    X = (X - X.mean(0)) / X.std(0)
    w = rng.normal(size=d)
    y = X @ w * 0.5 + np.tanh(X[:, 0] * X[:, 5]) + 0.5 * np.abs(X[:, 6]) + rng.normal(0.0, 0.3, size=n)
    y = (y - y.mean()) / y.std()
    return X.astype(np.float32), y.astype(np.float32)


def collider_shaped(seed=0):
    """10,000 x 28, two classes (about 47 / 53): standardised features whose class difference is
    a weak shift in a few coordinates plus a product term, so that a linear model gets about
    two thirds right (a hard, noisy binary problem of that shape)."""
    rng = np.random.default_rng(seed)
    n, d = 10000, 28
    X = rng.normal(size=(n, d))
    score = 0.6 * X[:, 0] - 0.5 * X[:, 3] + 0.7 * X[:, 1] * X[:, 2] + 0.4 * np.abs(X[:, 7]) + rng.normal(0.0, 1.0, size=n)
    y = (score > np.quantile(score, 0.47)).astype(np.float64)
    X = (X - X.mean(0)) / X.std(0)
    return X.astype(np.float32), y.astype(np.float32)


def workload(name, seed=0, n_configs=None, hidden=None, batch_size=None, epochs=None):
    """Named workloads.  Returns a dict with X, y, task, n_folds, configs, seed.

    ``iris8``      150x4x3,   8 configs (one suggest batch), 100 epochs
    ``breast128``  569x30x2,  128 configs (16 steps x 8),    200 epochs
    ``digits2048`` 1797x64x10, 2048 configs (16 studies x 128), 200 epochs
    ``diabetes4096`` 442x10 regression, 4096 configs (32 x 128), 200 epochs
    ``digits_sweep`` the digits shape with caller-chosen n_configs / hidden /
    batch_size (throughput sweep)
    ``housing10k`` 10000x8 regression, ``collider10k`` 10000x28x2: the 10,000-row shape of the
    paper's down-sampled sets, 128 configs, 50 epochs
    """
    table = {
        "iris8": (blobs_iris_shaped, TASK_CLASSIFICATION, 8, 100, 150),
        "breast128": (gaussians_breast_shaped, TASK_CLASSIFICATION, 128, 200, 150),
        "digits2048": (digits_shaped, TASK_CLASSIFICATION, 2048, 200, 250),
        "diabetes4096": (linear_diabetes_shaped, TASK_REGRESSION, 4096, 200, 250),
        "digits_sweep": (digits_shaped, TASK_CLASSIFICATION, 3200, 200, 250),
        "housing10k": (housing_shaped, TASK_REGRESSION, 128, 50, 250),
        "collider10k": (collider_shaped, TASK_CLASSIFICATION, 128, 50, 250),
    }
    gen, task, n_def, e_def, b_hi = table[name]
    X, y = gen(seed)
    configs = suggest_configs(
        n_def if n_configs is None else n_configs,
        seed + 1000,
        e_def if epochs is None else epochs,
        batch_hi=b_hi,
        hidden=hidden,
        batch_size=batch_size,
    )
    return dict(name=name, X=X, y=y, task=task, n_folds=5, configs=configs, seed=seed)
