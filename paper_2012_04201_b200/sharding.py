"""Splitting one ``params_list`` over several ranks (one process per GPU).

Every (configuration, fold) fit is independent and its random streams are keyed by the
configuration's position in the full list, so a rank that evaluates a subset and passes those
positions as keys (``bbo_mlp_cv_eval_keyed``; or, for a contiguous slice, the slice's first
position as ``config_index_base``) gets exactly the scores of the unsplit call.  No data-path
collective is involved; the scores are gathered at the end.  The paper deals independent jobs
to the GPUs in round-robin order (sec. 5); here the deal is balanced by estimated cost, because
the fits of one list differ tenfold in length.
"""
from __future__ import annotations

import numpy as np


def shard_bounds(n_configs: int, rank: int, world: int):
    """Contiguous slice [begin, end) of the list for ``rank``; the first ranks get one more."""
    if not (0 <= rank < world) or n_configs < 0:
        raise ValueError("bad rank/world/n_configs")
    base, rem = divmod(n_configs, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def config_costs(configs, n: int, d: int, n_classes: int, n_folds: int):
    """Estimated cost of each configuration (all its folds), in the units the library's launch
    order uses: per optimizer step a fixed part plus a part per hidden unit, and a part per
    training row and hidden unit; widths are scaled by (d + classes) relative to the 64-feature,
    10-class shape the constants were fitted on."""
    h = configs["hidden"].astype(np.float64) * (d + n_classes) / 74.0
    e = configs["epochs"].astype(np.float64)
    cost = np.zeros(configs.size, np.float64)
    for f in range(n_folds):
        n_tr = n - (n // n_folds + (1 if f < n % n_folds else 0))
        b = np.minimum(configs["batch_size"], n_tr).astype(np.float64)
        cost += e * np.ceil(n_tr / b) * (8000.0 + 80.0 * h) + e * n_tr * 2.9 * h
    return cost


def balanced_assignment(costs, world: int):
    """Rank of every list entry: entries in order of descending cost (ties: list order), each to
    the rank with the least cost so far (ties: lowest rank).  Deterministic, so every rank
    computes the same deal without communication."""
    costs = np.asarray(costs, np.float64)
    if world < 1:
        raise ValueError("world must be positive")
    assign = np.zeros(costs.size, np.int32)
    load = np.zeros(world, np.float64)
    for i in np.argsort(-costs, kind="stable"):
        r = int(np.argmin(load))
        assign[i] = r
        load[r] += costs[i]
    return assign


def shard_indices(assign, rank: int):
    """Positions (ascending) of the entries dealt to ``rank``."""
    return np.flatnonzero(np.asarray(assign) == rank).astype(np.int32)


def gather_scores(local_scores, n_configs: int, rank: int, world: int, dist=None):
    """All ranks' contiguous slices of scores (shard_bounds), concatenated in list order.
    ``dist``: torch.distributed (initialised), or None when world == 1.  Works with CPU (gloo)
    or CUDA (nccl) tensors."""
    import torch

    local = torch.as_tensor(local_scores, dtype=torch.float32)
    if world == 1:
        return local.clone()
    sizes = [shard_bounds(n_configs, r, world) for r in range(world)]
    longest = max(e - b for b, e in sizes)
    padded = torch.zeros(longest, dtype=torch.float32, device=local.device)
    padded[: local.numel()] = local
    parts = [torch.zeros_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    return torch.cat([parts[r][: e - b] for r, (b, e) in enumerate(sizes)])


def gather_scores_by_assignment(local_scores, assign, rank: int, world: int, dist=None):
    """Scores of the whole list, in list order, from every rank's scores of its own entries
    (``shard_indices(assign, rank)`` order).  One all-gather of the padded score vectors; every
    rank knows the deal, so no indices travel."""
    import torch

    assign = np.asarray(assign)
    local = torch.as_tensor(local_scores, dtype=torch.float32)
    if world == 1:
        return local.clone()
    counts = np.bincount(assign, minlength=world)
    padded = torch.zeros(int(counts.max()), dtype=torch.float32, device=local.device)
    padded[: local.numel()] = local
    parts = [torch.zeros_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    full = torch.zeros(assign.size, dtype=torch.float32, device=local.device)
    for r in range(world):
        idx = torch.as_tensor(shard_indices(assign, r).astype(np.int64), device=local.device)
        full[idx] = parts[r][: idx.numel()]
    return full
