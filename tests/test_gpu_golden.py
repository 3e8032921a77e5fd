"""Full-size parity against stored checker results.

The fold scores under ``tests/golden/*.npz`` were written by ``tests/golden/make_oracle_scores.py``
from the CPU checker alone (about two hours of CPU time, hence stored).  Here the CUDA path
evaluates the same configurations, keyed by their positions in the workload's list, and every
fold score is compared element by element: within 1e-3 absolute for at least 99 % of the fits
(the bar), and the fraction that is equal bit for bit is printed (the expectation: all).
"""
import os

import numpy as np
import pytest

from paper_2012_04201_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
SCORE_ATOL = 1e-3
SCORE_FRACTION = 0.99


def load_golden(name):
    path = os.path.join(GOLDEN, name + ".npz")
    if not os.path.exists(path):
        pytest.fail(f"{path} is missing: run tests/golden/make_oracle_scores.py {name}")
    z = np.load(path)
    return z["config_index"].astype(np.int32), z["fold_scores"].astype(np.float64), int(z["n_configs"])


def gpu_fold_scores(wl, idx):
    from paper_2012_04201_b200 import binding
    h = binding.MlpCv()
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    h.eval(X, y, wl["task"], wl["n_folds"], wl["configs"][idx], wl["seed"], config_keys=idx)
    fs = h.fold_scores().astype(np.float64)
    h.close()
    return fs


def compare(name, got, want):
    both_inf = np.isinf(got) & np.isinf(want) & (np.sign(got) == np.sign(want))
    err = np.where(both_inf, 0.0, np.abs(got - want))
    within = float(np.mean(err <= SCORE_ATOL))
    equal = float(np.mean((got == want) | both_inf))
    print(f"[{name}] fits={got.size} within_1e-3={within:.4f} bit_equal={equal:.4f} max_err={np.nanmax(err):.3g}")
    assert within >= SCORE_FRACTION
    return equal


@pytest.mark.parametrize("name,workload,kwargs", [
    ("diabetes4096_all", "diabetes4096", {}),
    ("housing10k_all", "housing10k", {}),
    ("digits2048_by_width", "digits2048", {}),
    ("digits_bench_cell", "digits_sweep", {"n_configs": 3200}),
])
def test_fold_scores_match_the_stored_checker_results(name, workload, kwargs):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    idx, want, n_configs = load_golden(name)
    wl = W.workload(workload, **kwargs)
    assert wl["configs"].size == n_configs
    got = gpu_fold_scores(wl, idx)
    assert got.shape == want.shape
    compare(name, got, want)
