"""The allocation-free entry point against the ordinary one.

``bbo_mlp_cv_eval_static`` is for callers that may not ask the driver for device memory
while they run (an arena allocator owns the heap, a latency-bound loop cannot afford
cudaMalloc's implicit synchronisation, or no free memory is left).  It keeps all of its
working memory in one fixed array inside the library, which every call reuses.  The test
therefore calls it twice in a row -- the second call starts from the first call's leftovers --
with different inputs, and checks each result against ``bbo_mlp_cv_eval`` and against the CPU
checker, and that the device's free memory is the same before and after a call.

Collected last on purpose (file name), and self-contained: it passes alone in a fresh
process and after the rest of the suite.
"""
import numpy as np
import pytest

import oracle
from paper_2012_04201_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SCORE_ATOL = 1e-3


def reference_scores(binding, wl, cfg):
    h = binding.MlpCv()
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    s = h.eval(X, y, wl["task"], wl["n_folds"], cfg, wl["seed"]).cpu().numpy()
    h.close()
    return s


def static_scores(binding, wl, cfg, n_classes=0):
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    out = torch.full((cfg.size,), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    rc = binding.bbo_mlp_cv_eval_static(stream, X.data_ptr(), y.data_ptr(), X.shape[0], X.shape[1], wl["task"],
                                        wl["n_folds"], n_classes, cfg, wl["seed"], out.data_ptr())
    assert rc == binding.BBO_OK, rc
    return out.cpu().numpy()


def test_static_entry_point_matches_eval_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2012_04201_b200 import binding

    # first call: classification, d = 30 (rows need no padding), 12 configurations
    a = W.workload("breast128", n_configs=12, epochs=6)
    # second call: regression, d = 7 (padded copy of X goes through the fixed array), fewer
    # and smaller fits, so stale fit-list and score entries of the first call remain behind it
    b = W.workload("diabetes4096", n_configs=5, epochs=9)
    b["X"] = np.ascontiguousarray(b["X"][:, :7])
    got_a = static_scores(binding, a, a["configs"])   # also the warm-up: kernels of both shapes get loaded
    got_b = static_scores(binding, b, b["configs"])
    # the property in the name: a call leaves the device's free memory where it found it
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    got_a2 = static_scores(binding, a, a["configs"], n_classes=2)
    got_b2 = static_scores(binding, b, b["configs"])
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    want_a = reference_scores(binding, a, a["configs"])
    want_b = reference_scores(binding, b, b["configs"])
    for got, want in ((got_a, want_a), (got_b, want_b), (got_a2, want_a), (got_b2, want_b)):
        assert np.all(np.isfinite(got))
        assert np.max(np.abs(got - want)) <= SCORE_ATOL
    print("static vs eval bit-equal:", np.array_equal(got_a, want_a), np.array_equal(got_b, want_b))
    # and against the CPU checker, which shares nothing with the CUDA path
    for wl, got in ((a, got_a2), (b, got_b2)):
        ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], wl["n_folds"], wl["configs"], wl["seed"])["scores"]
        assert np.mean(np.abs(got.astype(np.float64) - ref) <= SCORE_ATOL) >= 0.99
        print("static vs checker bit-equal:", np.array_equal(got.astype(np.float64), ref))
    assert binding.load().bbo_mlp_cv_static_last_cuda_error() == b""


def test_static_entry_point_rejects_oversized_problems():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2012_04201_b200 import binding

    wl = W.workload("iris8")
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    many = W.suggest_configs(4097, 1, 1)
    out = torch.empty(4097, dtype=torch.float32, device="cuda")
    rc = binding.bbo_mlp_cv_eval_static(0, X.data_ptr(), y.data_ptr(), 150, 4, 0, 5, 0, many, 0, out.data_ptr())
    assert rc == binding.BBO_ERR_TOO_LARGE
    assert b"fixed scratch" in binding.load().bbo_mlp_cv_strerror(rc)
    big = torch.zeros(5000, 4, device="cuda")
    yb = torch.zeros(5000, device="cuda")
    rc = binding.bbo_mlp_cv_eval_static(0, big.data_ptr(), yb.data_ptr(), 5000, 4, 1, 5, 0, wl["configs"], 0,
                                        out.data_ptr())
    assert rc == binding.BBO_ERR_TOO_LARGE
