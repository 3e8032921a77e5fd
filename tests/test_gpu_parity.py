"""CUDA path against the CPU checker, through the C ABI, on the same seeded inputs.

Bars: random words, exponential, fold split and minibatch order bit-exact; training loss of
the first 50 optimizer steps within 1e-4 relative; held-out fold score within 1e-3 absolute
for at least 99 % of fits (the arithmetic order is fixed on both sides, so the scores are
expected to be equal bit for bit and the tests report whether they are).
"""
import numpy as np
import pytest

import oracle
from paper_2012_04201_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

LOSS_RTOL = 1e-4
SCORE_ATOL = 1e-3
SCORE_FRACTION = 0.99


@pytest.fixture(scope="module")
def binding():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2012_04201_b200 import binding as b
    return b


def gpu_eval(binding, wl, configs, trace_steps=0, keep_theta=False, seed=None, n_folds=None):
    h = binding.MlpCv(trace_steps=trace_steps, keep_theta=keep_theta)
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    K = wl["n_folds"] if n_folds is None else n_folds
    scores = h.eval(X, y, wl["task"], K, configs, wl["seed"] if seed is None else seed).cpu().numpy()
    out = dict(scores=scores, fold_scores=h.fold_scores())
    if trace_steps:
        out["trace"] = h.loss_trace()
    if keep_theta:
        c = configs[-1]
        C = 1 if wl["task"] == 1 else int(wl["y"].max()) + 1
        out["theta"] = h.debug_theta(oracle.param_count(wl["X"].shape[1], int(c["hidden"]), C))
    h.close()
    return out


def check_against_oracle(gpu, ref, label):
    fs_g, fs_r = gpu["fold_scores"].astype(np.float64), ref["fold_scores"]
    both_inf = np.isinf(fs_g) & np.isinf(fs_r) & (np.sign(fs_g) == np.sign(fs_r))
    err = np.where(both_inf, 0.0, np.abs(fs_g - fs_r))
    frac = np.mean(err <= SCORE_ATOL)
    exact = np.mean((fs_g == fs_r) | both_inf)
    print(f"[{label}] fits={fs_g.size} within_1e-3={frac:.4f} bit_equal={exact:.4f} max_err={np.nanmax(err):.3g}")
    assert frac >= SCORE_FRACTION
    m_g, m_r = gpu["scores"].astype(np.float64), ref["scores"]
    ok = np.isinf(m_g) & np.isinf(m_r) | (np.abs(m_g - m_r) <= SCORE_ATOL)
    assert np.mean(ok) >= SCORE_FRACTION
    if "trace" in gpu and ref.get("trace") is not None:
        tg, tr = gpu["trace"].astype(np.float64), ref["trace"]
        assert np.array_equal(np.isnan(tg), np.isnan(tr))
        fin = np.isfinite(tr) & np.isfinite(tg)
        rel = np.abs(tg[fin] - tr[fin]) / np.maximum(np.abs(tr[fin]), 1e-30)
        print(f"[{label}] loss trace: max rel err {rel.max():.3g} over {fin.sum()} steps")
        assert rel.max() <= LOSS_RTOL
        assert np.array_equal(np.isinf(tg), np.isinf(tr))
    return exact


def test_random_words_bit_exact(binding):
    rng = np.random.default_rng(0)
    N = 1_000_000
    ctr = np.stack([rng.integers(0, 16, N), rng.integers(0, 2**32, N), rng.integers(0, 2**32, N),
                    rng.integers(0, 2**28, N), rng.integers(0, 2**32, N)], 1).astype(np.uint32)
    ctr[:4] = [[1, 0, 0, 0, 0], [15, 2**32 - 1, 2**32 - 1, 2**28 - 1, 2**32 - 1], [3, 0, 2**32 - 1, 0, 1], [2, 7, 4, 3, 0]]
    h = binding.MlpCv()
    for seed in (0, 2**64 - 1, 0x0123456789ABCDEF):
        assert np.array_equal(h.debug_rng(seed, ctr), oracle.rng_blocks(seed, ctr))
    h.close()


def test_exponential_bit_exact(binding):
    x = np.concatenate([np.linspace(-90.0, 0.0, 1_000_001), -np.logspace(-12, 2, 200_001),
                        np.linspace(0.0, 90.0, 100_001), [np.nan, -np.inf, np.inf, -0.0]]).astype(np.float32)
    h = binding.MlpCv()
    got, want = h.debug_exp(x), oracle.expf_array(x)
    h.close()
    assert np.array_equal(got.view(np.uint32)[:-4], want.view(np.uint32)[:-4])
    assert np.isnan(got[-4]) and got[-3] == 0.0 and np.isinf(got[-2]) and got[-1] == 1.0


def test_branch_free_sqrt_and_division_equal_ieee(binding):
    h = binding.MlpCv()
    # every non-negative float bit pattern (zero, denormals, normals, inf, NaN): the fast path
    # must agree with the IEEE square root wherever it claims to be valid
    out = h.debug_fast_math(0, first=0, count=2**31)
    assert out[0] == 0 and out[1] > 1.3e9, out
    # 2^32 operand triples with exponents across the whole range
    total_safe = 0
    for seed in (1, 2):
        out = h.debug_fast_math(1, seed=seed, count=2**31)
        assert out[0] == 0, out
        total_safe += int(out[1])
    assert total_safe > 5e7
    # tiny and denormal first moments over ordinary denominators: denormal quotients, which long
    # fits with an L2 term produce all the time, must come out of the fast path, and exactly
    for seed in (4, 5):
        out = h.debug_fast_math(3, seed=seed, count=2**31)
        assert out[0] == 0, out
        assert out[1] > 0.9 * 2**31, out
    # softmax quotients: exponentials of non-positive numbers over denominators in [1, 16]
    out = h.debug_fast_math(2, seed=3, count=2**30)
    assert out[0] == 0 and out[1] > 1.0e9, out
    h.close()


@pytest.mark.parametrize("n,K", [(150, 5), (569, 5), (1797, 5), (442, 5), (37, 3), (12, 12), (4100, 7)])
def test_fold_split_and_minibatch_order_bit_exact(binding, n, K):
    h = binding.MlpCv()
    for seed, config, fold, epoch in [(0, 0, 0, 0), (0, 5, K - 1, 199), (123456789012345, 2047, 1, 17)]:
        fo, order = h.debug_indices(n, K, seed, config, fold, epoch)
        _, fo_ref = oracle.fold_split(n, K, seed)
        assert np.array_equal(fo, fo_ref)
        assert np.array_equal(order, oracle.epoch_order(n, K, seed, config, fold, epoch))
    h.close()


def test_iris_shaped_all_fits(binding):
    wl = W.workload("iris8")
    gpu = gpu_eval(binding, wl, wl["configs"], trace_steps=50, keep_theta=True)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"], trace_steps=50)
    exact = check_against_oracle(gpu, ref, "iris8")
    th = oracle.cv_fits(wl["X"], wl["y"], 0, 5, wl["configs"], 0, [7], [4], want_theta=True)["theta"]
    print("[iris8] final parameters bit-equal:", np.array_equal(gpu["theta"].astype(np.float64), th))
    np.testing.assert_allclose(gpu["theta"], th, rtol=1e-3, atol=1e-4)
    assert exact >= 0.9


def test_breast_shaped_all_fits(binding):
    wl = W.workload("breast128")
    gpu = gpu_eval(binding, wl, wl["configs"], trace_steps=50)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"], trace_steps=50)
    check_against_oracle(gpu, ref, "breast128")


def test_diabetes_shaped_subset(binding):
    wl = W.workload("diabetes4096", n_configs=160)
    gpu = gpu_eval(binding, wl, wl["configs"], trace_steps=50)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"], trace_steps=50)
    check_against_oracle(gpu, ref, "diabetes160")
    assert np.all(gpu["fold_scores"] <= 0.0)


def test_digits_shaped_short_and_full_length(binding):
    # many fits with few epochs (several sub-tiles, ragged last batch), a few at full length
    wl = W.workload("digits2048", n_configs=48, epochs=6)
    gpu = gpu_eval(binding, wl, wl["configs"], trace_steps=50, keep_theta=True)
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"], trace_steps=50)
    check_against_oracle(gpu, ref, "digits48x6ep")
    th = oracle.cv_fits(wl["X"], wl["y"], 0, 5, wl["configs"], 0, [47], [4], want_theta=True)["theta"]
    print("[digits] final parameters bit-equal:", np.array_equal(gpu["theta"].astype(np.float64), th))
    wl = W.workload("digits2048", n_configs=4)
    gpu = gpu_eval(binding, wl, wl["configs"])
    ref = oracle.cv_eval(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"])
    check_against_oracle(gpu, ref, "digits4x200ep")


def make_configs(rows):
    c = np.zeros(len(rows), W.CONFIG_DTYPE)
    for i, r in enumerate(rows):
        c[i] = r
    return c


def test_edge_cases(binding):
    wl = W.workload("iris8")
    cfg = make_configs([
        (1, 7, 3, 0.0, 1e-2, 0.9, 0.999, 1e-8),       # one hidden unit, ragged batches
        (200, 1, 1, 1e-3, 1e-3, 0.5, 0.9, 1e-6),      # batch of one row
        (50, 1000, 5, 10.0, 1e-1, 0.0, 0.0, 1e-9),    # batch above the fold size, zero betas
        (64, 33, 0, 1e-4, 1e-3, 0.9, 0.999, 1e-8),    # zero epochs: scores the initial weights
        (57, 120, 4, 1e-5, 0.0, 0.9, 0.999, 1e-8),    # lr = 0
        (13, 31, 9, 1e-2, 1e-1, 0.99, 0.999999, 1e-9),
    ])
    gpu = gpu_eval(binding, wl, cfg, trace_steps=50)
    ref = oracle.cv_eval(wl["X"], wl["y"], 0, 5, cfg, 0, trace_steps=50)
    check_against_oracle(gpu, ref, "edge-iris")
    # leave-one-out on a tiny set, two classes, and a 2-fold split
    tiny = dict(X=wl["X"][:12].copy(), y=(wl["y"][:12] > 0).astype(np.float32), task=0, n_folds=12, seed=3)
    gpu = gpu_eval(binding, tiny, cfg[:3])
    ref = oracle.cv_eval(tiny["X"], tiny["y"], 0, 12, cfg[:3], 3)
    check_against_oracle(gpu, ref, "edge-loo")
    gpu = gpu_eval(binding, wl, cfg[:2], n_folds=2, seed=11)
    ref = oracle.cv_eval(wl["X"], wl["y"], 0, 2, cfg[:2], 11)
    check_against_oracle(gpu, ref, "edge-2fold")
    # regression with d not a multiple of four and a diverging learning rate
    wr = W.workload("diabetes4096", n_configs=2)
    X = np.ascontiguousarray(wr["X"][:, :7])
    cfg = make_configs([(20, 16, 30, 0.0, 0.1, 0.9, 0.9, 1e-9), (9, 5, 3, 1.0, 1e-3, 0.9, 0.99, 1e-8)])
    w2 = dict(X=X, y=wr["y"], task=1, n_folds=5, seed=0)
    gpu = gpu_eval(binding, w2, cfg, trace_steps=50)
    ref = oracle.cv_eval(X, wr["y"], 1, 5, cfg, 0, trace_steps=50)
    check_against_oracle(gpu, ref, "edge-reg-d7")


def test_weights_that_decay_into_denormals_stay_bit_equal(binding):
    # Two constant-zero feature columns: their weights see only the L2 term, decay geometrically
    # and end up denormal together with their gradients and first moments, so m / (sqrt(v) + eps)
    # is denormal for most of the fit.  The update's fast path must give the IEEE quotient there.
    wl = W.workload("iris8")
    X = np.concatenate([wl["X"], np.zeros((wl["X"].shape[0], 2), np.float32)], axis=1)
    cfg = make_configs([
        (16, 16, 150, 1e-2, 1e-3, 0.9, 0.999, 1e-8),
        (24, 8, 400, 1e-1, 3e-3, 0.9, 0.999, 1e-8),
        (40, 16, 400, 1e-1, 1e-2, 0.9, 0.999, 1e-8),
    ])
    for task, y in ((0, wl["y"]), (1, wl["X"][:, 0].copy())):   # classification and regression kernels
        w2 = dict(X=X, y=y, task=task, n_folds=5, seed=5)
        gpu = gpu_eval(binding, w2, cfg, keep_theta=True)
        ref = oracle.cv_eval(X, y, task, 5, cfg, 5)
        exact = check_against_oracle(gpu, ref, f"denormal-task{task}")
        th = oracle.cv_fits(X, y, task, 5, cfg, 5, [2], [4], want_theta=True)["theta"]
        w1 = th[: 6 * 40].reshape(6, 40)[4:]                    # weights of the two zero columns
        tiny = np.abs(w1[w1 != 0.0]) < 1.1754944e-38
        print(f"[denormal-task{task}] zero-column weights: {tiny.sum()} of {w1.size} denormal, bit-equal parameters:",
              np.array_equal(gpu["theta"].astype(np.float64), th))
        assert tiny.sum() + np.sum(w1 == 0.0) >= w1.size // 2      # the regime is actually reached
        assert np.array_equal(gpu["theta"].astype(np.float64), th)
        assert exact == 1.0


def test_score_depends_only_on_own_config_and_is_deterministic(binding):
    wl = W.workload("breast128", n_configs=12, epochs=8)
    a = gpu_eval(binding, wl, wl["configs"])
    b = gpu_eval(binding, wl, wl["configs"])
    assert np.array_equal(a["fold_scores"], b["fold_scores"])
    sub = wl["configs"][:5].copy()
    sub[0] = wl["configs"][9]
    c = gpu_eval(binding, wl, sub)
    assert np.array_equal(c["fold_scores"][1:5], a["fold_scores"][1:5])
    # host-buffer entry point gives the same scores
    h = binding.MlpCv()
    s = h.eval_host(wl["X"], wl["y"], wl["task"], 5, wl["configs"], wl["seed"])
    h.close()
    assert np.array_equal(s, a["scores"])


def test_error_codes(binding):
    wl = W.workload("iris8")
    h = binding.MlpCv()
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    bad = wl["configs"].copy()
    bad["beta1"][0] = 1.0
    with pytest.raises(binding.BboError) as e:
        h.eval(X, y, 0, 5, bad, 0)
    assert e.value.code == binding.BBO_ERR_INVALID_ARG
    with pytest.raises(binding.BboError):
        h.eval(X, y, 0, 1, wl["configs"], 0)           # one fold
    with pytest.raises(binding.BboError):
        h.eval(X, y - 0.5, 0, 5, wl["configs"], 0)     # fractional labels
    big = wl["configs"].copy()
    big["hidden"][0] = 100000
    with pytest.raises(binding.BboError) as e:
        h.eval(X, y, 0, 5, big, 0)
    assert e.value.code == binding.BBO_ERR_UNSUPPORTED
    # a shape over the caps is turned away before any scratch is reserved for it
    free0 = torch.cuda.mem_get_info()[0]
    wide = torch.zeros(16, 100000, device="cuda")
    yw = torch.zeros(16, device="cuda")
    free1 = torch.cuda.mem_get_info()[0]
    with pytest.raises(binding.BboError) as e:
        h.eval(wide, yw, 1, 2, wl["configs"], 0)
    assert e.value.code == binding.BBO_ERR_UNSUPPORTED
    assert torch.cuda.mem_get_info()[0] == free1
    del wide, yw, free0
    out = torch.empty(8, device="cuda")
    rc = binding.bbo_mlp_cv_eval(h._h, wl["X"].ctypes.data, y.data_ptr(), 150, 4, 0, 5, wl["configs"], 0, out.data_ptr())
    assert rc == binding.BBO_ERR_INVALID_ARG           # host pointer where a device pointer is required
    # the handle stays usable after errors
    s = h.eval(X, y, 0, 5, wl["configs"], 0)
    assert torch.isfinite(s).all()
    caps = h.query_caps(64, 10)
    assert caps["max_hidden"] >= 200 and caps["max_classes"] >= 10
    h.close()


def test_split_list_with_index_base_equals_unsplit_call(binding):
    from paper_2012_04201_b200 import sharding
    wl = W.workload("breast128", n_configs=11, epochs=5)
    whole = gpu_eval(binding, wl, wl["configs"])
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    parts = []
    for rank in range(3):
        b, e = sharding.shard_bounds(11, rank, 3)
        h = binding.MlpCv(config_index_base=b)
        parts.append(h.eval(X, y, wl["task"], 5, wl["configs"][b:e], wl["seed"]).cpu().numpy())
        h.close()
    assert np.array_equal(np.concatenate(parts), whole["scores"])


def test_cost_balanced_split_with_keys_equals_unsplit_call(binding):
    """One list dealt to three handles by estimated cost, every entry keyed by its position in
    the unsplit list (the multi-GPU path of bench.py, here on one GPU)."""
    from paper_2012_04201_b200 import sharding
    wl = W.workload("digits2048", n_configs=13, epochs=3)
    whole = gpu_eval(binding, wl, wl["configs"])
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    assign = sharding.balanced_assignment(sharding.config_costs(wl["configs"], 1797, 64, 10, 5), 3)
    full = np.full(13, np.nan, np.float32)
    for rank in range(3):
        mine = sharding.shard_indices(assign, rank)
        h = binding.MlpCv(config_index_base=1000)   # ignored by the keyed call
        full[mine] = h.eval(X, y, wl["task"], 5, wl["configs"][mine], wl["seed"], config_keys=mine).cpu().numpy()
        h.close()
    assert np.array_equal(full, whole["scores"])
    h = binding.MlpCv()
    with pytest.raises(binding.BboError) as e:
        h.eval(X, y, wl["task"], 5, wl["configs"][:2], wl["seed"], config_keys=np.array([0, -1], np.int32))
    assert e.value.code == binding.BBO_ERR_INVALID_ARG
    h.close()


def test_variant_option(binding):
    h = binding.MlpCv(variant=binding.VARIANT_FP32)
    h.close()
    with pytest.raises(binding.BboError) as e:
        binding.MlpCv(variant=binding.VARIANT_TF32)      # named in the header, not built
    assert e.value.code == binding.BBO_ERR_UNSUPPORTED
    with pytest.raises(binding.BboError) as e:
        binding.MlpCv(variant=7)
    assert e.value.code == binding.BBO_ERR_INVALID_ARG


def test_register_fma_rate_is_near_the_nominal_peak(binding):
    h = binding.MlpCv()
    tf = h.debug_ffma_peak()
    h.close()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nominal = sms * 128 * 2 * 1.965e9 / 1e12
    assert 0.6 * nominal < tf < 1.05 * nominal, tf


def test_bench_workload_sampled_fits_match_oracle(binding):
    """The launch configuration bench.py times (digits-shaped sweep, 4,000 fits, mixed widths
    and batch sizes, 200 epochs), with a sample of whole fits recomputed by the checker."""
    wl = W.workload("digits_sweep", seed=0, n_configs=800, epochs=200)
    gpu = gpu_eval(binding, wl, wl["configs"])
    assert np.all(np.isfinite(gpu["fold_scores"])) and gpu["fold_scores"].min() >= 0 and gpu["fold_scores"].max() <= 1
    cfg = wl["configs"]
    cost = cfg["hidden"].astype(np.float64)                      # cheap fits dominate the sample
    order = np.argsort(cost)
    pick = np.concatenate([order[:12], order[len(order) // 2: len(order) // 2 + 3], order[-1:]])
    rng = np.random.default_rng(0)
    fc = pick.astype(np.int32)
    ff = rng.integers(0, 5, size=fc.size).astype(np.int32)
    ref = oracle.cv_fits(wl["X"], wl["y"], wl["task"], 5, cfg, wl["seed"], fc, ff)["scores"]
    got = gpu["fold_scores"][fc, ff].astype(np.float64)
    print("[bench workload] sampled fits:", fc.size, "bit-equal:", int(np.sum(got == ref)))
    assert np.mean(np.abs(got - ref) <= SCORE_ATOL) >= SCORE_FRACTION
    m = gpu["fold_scores"].astype(np.float32)
    mean = ((((m[:, 0] + m[:, 1]) + m[:, 2]) + m[:, 3]) + m[:, 4]) / np.float32(5)
    assert np.array_equal(mean, gpu["scores"])


def test_batched_studies_on_the_device_follow_the_checker(binding):
    """Algorithm 1 with the device evaluation: several studies advance in lockstep, one call per
    iteration; because scores are bit-equal to the checker's, the trajectories are identical."""
    from paper_2012_04201_b200 import driver
    wl = W.workload("iris8")
    X = torch.from_numpy(wl["X"]).cuda()
    y = torch.from_numpy(wl["y"]).cuda()
    h = binding.MlpCv()

    def make():
        return [[driver.RandomSearch(10 + s, 12), driver.LocalPerturbation(20 + s, 12)] for s in range(3)]

    dev = driver.run_studies(lambda c, sizes: h.eval(X, y, 0, 5, c, 0).cpu().numpy(), make(), n_step=3, n_batch=8)
    ref = driver.run_studies(lambda c, sizes: oracle.cv_eval(wl["X"], wl["y"], 0, 5, c, 0)["scores"], make(),
                             n_step=3, n_batch=8)
    h.close()
    for ld, lr in zip(dev, ref):
        for (cd, sd), (cr, sr) in zip(ld, lr):
            assert np.array_equal(cd, cr) and np.array_equal(sd, sr)
