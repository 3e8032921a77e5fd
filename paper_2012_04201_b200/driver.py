"""Suggest-observe loops around the evaluation (paper, Algorithm 1).

Left algorithm: one optimizer suggests ``n_batch`` configurations per iteration, the
evaluation returns their cross-validation scores, the optimizer observes them; ``n_step``
iterations (the paper's runs use N_STEP = 16, N_BATCH = 8, sec. 2).  Right algorithm: two
optimizers each suggest ``n_batch / 2``, the lists are concatenated and evaluated together,
and both optimizers observe all scores (sec. 4).

The optimizers here are two small self-contained ones (random search and a local perturbation
search); the paper's third-party optimizers are out of scope.  What this module shows is how
the evaluation is driven: ``run_studies`` advances many independent studies in lockstep and
sends all their suggestions of one iteration to the device in a single call, which is how
thousands of fits end up in one launch.  Scores follow the library's convention (higher is
better); Bayesmark minimises a loss, i.e. the negated score.
"""
from __future__ import annotations

import numpy as np

from .workloads import CONFIG_DTYPE

#: search space of the MLP-adam configurations (log10 ranges for the log-uniform fields)
SPACE = {
    "hidden": ("int", 50, 200),
    "batch_size": ("int", 10, 250),
    "alpha": ("log", -5.0, 1.0),
    "lr": ("log", -5.0, -1.0),
    "beta1": ("lin", 0.5, 0.99),
    "beta2": ("lin", 0.9, 0.999999),
    "eps": ("log", -9.0, -6.0),
}
_FIELDS = list(SPACE)


def _to_unit(configs):
    """Configurations -> points of the unit cube (one coordinate per searched field)."""
    u = np.zeros((configs.size, len(_FIELDS)))
    for k, name in enumerate(_FIELDS):
        kind, lo, hi = SPACE[name]
        v = configs[name].astype(np.float64)
        if kind == "log":
            v = np.log10(v)
        u[:, k] = (v - lo) / (hi - lo)
    return np.clip(u, 0.0, 1.0)


def _from_unit(u, epochs):
    """Points of the unit cube -> configurations."""
    out = np.zeros(u.shape[0], dtype=CONFIG_DTYPE)
    for k, name in enumerate(_FIELDS):
        kind, lo, hi = SPACE[name]
        v = lo + np.clip(u[:, k], 0.0, 1.0) * (hi - lo)
        if kind == "int":
            out[name] = np.rint(v).astype(np.int32)
        elif kind == "log":
            out[name] = (10.0 ** v).astype(np.float32)
        else:
            out[name] = v.astype(np.float32)
    out["beta2"] = np.minimum(out["beta2"], np.float32(0.99999994))
    out["epochs"] = epochs
    return out


class RandomSearch:
    """Uniform samples of the search space."""

    def __init__(self, seed, epochs):
        self.rng = np.random.default_rng(seed)
        self.epochs = epochs
        self.history = []

    def suggest(self, n):
        return _from_unit(self.rng.uniform(size=(n, len(_FIELDS))), self.epochs)

    def observe(self, configs, scores):
        self.history.append((configs.copy(), np.asarray(scores, np.float64).copy()))


class LocalPerturbation:
    """Keeps the best configuration seen so far (by any optimizer whose observations it is
    given) and suggests Gaussian perturbations of it in the unit cube, with a radius that
    shrinks as iterations pass; the first iteration is random."""

    def __init__(self, seed, epochs, radius=0.25, decay=0.85):
        self.rng = np.random.default_rng(seed)
        self.epochs = epochs
        self.radius = radius
        self.decay = decay
        self.best_u = None
        self.best_score = -np.inf

    def suggest(self, n):
        if self.best_u is None:
            u = self.rng.uniform(size=(n, len(_FIELDS)))
        else:
            u = self.best_u[None, :] + self.rng.normal(0.0, self.radius, size=(n, len(_FIELDS)))
        return _from_unit(u, self.epochs)

    def observe(self, configs, scores):
        scores = np.asarray(scores, np.float64)
        finite = np.where(np.isfinite(scores), scores, -np.inf)
        i = int(np.argmax(finite))
        if finite[i] > self.best_score:
            self.best_score = float(finite[i])
            self.best_u = _to_unit(configs[i:i + 1])[0]
        self.radius *= self.decay


def run_study(evaluate, optimizers, n_step=16, n_batch=8):
    """Algorithm 1 for one study.  ``optimizers``: one optimizer (left algorithm) or two (right
    algorithm: each suggests n_batch / 2, both observe everything).  ``evaluate(configs)``
    returns one score per configuration.  Returns the list of (configs, scores) per iteration."""
    return run_studies(lambda cfgs, _sizes: evaluate(cfgs), [optimizers], n_step, n_batch)[0]


def run_studies(evaluate, studies, n_step=16, n_batch=8):
    """Advances several independent studies in lockstep.  ``studies``: list whose entries are
    one optimizer or a pair of optimizers.  Per iteration the suggestions of all studies are
    concatenated (study-major) and evaluated by ONE call ``evaluate(configs, sizes)``, where
    ``sizes[i]`` is the number of configurations of study i; the scores are split back and
    observed.  Returns, per study, the list of (configs, scores) per iteration."""
    studies = [list(s) if isinstance(s, (list, tuple)) else [s] for s in studies]
    for opts in studies:
        if len(opts) not in (1, 2) or n_batch % len(opts) != 0:
            raise ValueError("a study has one optimizer, or two with an even n_batch")
    logs = [[] for _ in studies]
    for _ in range(n_step):
        per_study = []
        for opts in studies:
            share = n_batch // len(opts)
            per_study.append(np.concatenate([o.suggest(share) for o in opts]))
        sizes = [c.size for c in per_study]
        scores = np.asarray(evaluate(np.concatenate(per_study), sizes), np.float64)
        if scores.shape[0] != sum(sizes):
            raise ValueError("evaluate must return one score per configuration")
        off = 0
        for opts, cfgs, log in zip(studies, per_study, logs):
            s = scores[off:off + cfgs.size]
            off += cfgs.size
            for o in opts:           # every optimizer of the study observes all of its scores
                o.observe(cfgs, s)
            log.append((cfgs, s))
    return logs


def best_so_far(log):
    """Running maximum of the scores of a study's log (one value per iteration)."""
    best, out = -np.inf, []
    for _, s in log:
        s = np.where(np.isfinite(s), s, -np.inf)
        best = max(best, float(s.max()))
        out.append(best)
    return out
