"""Writes the stored fold scores that the full-size GPU parity tests compare against.

Every value comes from the CPU checker (``oracle/``) on the seeded synthetic workloads of
``paper_2012_04201_b200/workloads.py``; nothing here touches the CUDA library.  The checker
needs about two hours of CPU time for all four files, which is why its results are stored:

  diabetes4096_all.npz       every fit of the diabetes-shaped workload (4096 configurations x 5 folds)
  digits2048_by_width.npz    digits-shaped workload, 200 epochs: for each padded hidden width
                             56, 64, ..., 200 six configurations spread over the batch sizes
  digits_bench_cell.npz      the benchmark's default workload (3200 configurations, 16,000 fits):
                             104 configurations evenly spaced in the order of estimated cost
  housing10k_all.npz         the 10,000-row regression workload at its full 50 epochs

Each file holds ``config_index`` (positions in the workload's configuration list, which key the
random streams) and ``fold_scores`` [len(config_index), 5] as the checker's float results.

Usage:  python tests/golden/make_oracle_scores.py [--threads N] [name ...]
Existing files are kept unless named explicitly.
"""
from __future__ import annotations

import argparse
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2012_04201_b200 import workloads as W  # noqa: E402

BENCH_CONFIGS = 3200  # 16,000 fits: the benchmark's default workload


def estimated_cost(configs, n_train):
    """Relative cost of a fit: rows visited times width, plus a per-step term."""
    h = configs["hidden"].astype(np.float64)
    b = np.minimum(configs["batch_size"], n_train).astype(np.float64)
    steps = configs["epochs"] * np.ceil(n_train / b)
    return configs["epochs"] * n_train * h + steps * 30.0 * h


def pick_by_width(configs, per_width=6):
    """For every padded hidden width, `per_width` configurations spread over the batch sizes."""
    padded = (configs["hidden"] + 7) // 8 * 8
    chosen = []
    for w in range(56, 201, 8):
        idx = np.flatnonzero(padded == w)
        idx = idx[np.argsort(configs["batch_size"][idx], kind="stable")]
        take = np.unique(np.round(np.linspace(0, idx.size - 1, per_width)).astype(int))
        chosen.extend(idx[take].tolist())
    return np.array(sorted(chosen), np.int32)


def pick_by_cost(configs, n_train, count):
    order = np.argsort(estimated_cost(configs, n_train), kind="stable")
    take = np.unique(np.round(np.linspace(0, order.size - 1, count)).astype(int))
    return np.sort(order[take]).astype(np.int32)


def selections():
    """name -> (workload dict, config indices)."""
    out = {}
    wl = W.workload("diabetes4096")
    out["diabetes4096_all"] = (wl, np.arange(wl["configs"].size, dtype=np.int32))
    wl = W.workload("housing10k")
    out["housing10k_all"] = (wl, np.arange(wl["configs"].size, dtype=np.int32))
    wl = W.workload("digits2048")
    out["digits2048_by_width"] = (wl, pick_by_width(wl["configs"]))
    wl = W.workload("digits_sweep", n_configs=BENCH_CONFIGS)
    out["digits_bench_cell"] = (wl, pick_by_cost(wl["configs"], 1438, 104))
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("names", nargs="*")
    args = ap.parse_args()
    sel = selections()
    for name, (wl, idx) in sel.items():
        path = os.path.join(HERE, name + ".npz")
        if args.names and name not in args.names:
            continue
        if not args.names and os.path.exists(path):
            continue
        K = wl["n_folds"]
        fit_config = np.repeat(idx, K).astype(np.int32)
        fit_fold = np.tile(np.arange(K, dtype=np.int32), idx.size)
        t0 = time.time()
        res = oracle.cv_fits(wl["X"], wl["y"], wl["task"], K, wl["configs"], wl["seed"], fit_config, fit_fold,
                             n_threads=args.threads)
        fs = res["scores"].reshape(idx.size, K)
        np.savez_compressed(path, config_index=idx, fold_scores=fs, workload=np.array(wl["name"]),
                            n_configs=np.array(wl["configs"].size), seed=np.array(wl["seed"]))
        print(f"{name}: {fs.size} fits in {time.time() - t0:.0f} s -> {path}", flush=True)


if __name__ == "__main__":
    main()
