"""CPU checker (ctypes wrapper).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may
import this package.  The CUDA library and its Python binding never do; neither imports
the other.  The arithmetic lives in ``mlp_cv_oracle.cpp`` (see its header for what it
follows in the paper and how it is pinned).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mlp_cv_oracle.cpp")
_LIB = os.path.join(_HERE, "libmlp_cv_oracle.so")

MODE_F32 = 0
MODE_F64 = 1
MODE_F32_TF32_OPERANDS = 2   # experiment: operands of the two large contractions rounded to TF32
MODE_F32_BLOCKED = 3         # experiment: exact float products, summed in blocks of 8 as a matrix unit would
MODE_F32_BLOCKED_SPLIT = 4   # experiment: the blocked order with hi/lo TF32 operand splits (three products per term)
STREAM_FOLD, STREAM_INIT, STREAM_PERM = 1, 2, 3
SOLVER_ADAM, SOLVER_SGD = 0, 1
METRIC_DEFAULT, METRIC_ALT = 0, 1   # accuracy / -MSE, or -NLL / -MAE

CONFIG_DTYPE = np.dtype(
    [("hidden", "<i4"), ("batch_size", "<i4"), ("epochs", "<i4"), ("alpha", "<f4"),
     ("lr", "<f4"), ("beta1", "<f4"), ("beta2", "<f4"), ("eps", "<f4")]
)


def build(force: bool = False) -> str:
    """Compile the checker with g++ (no fast-math, no implicit contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-ffp-contract=off", "-mfma", "-fopenmp", "-shared", "-fPIC",
               "-std=c++17", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32, u64, i32, i64, f64 = (ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32,
                                   ctypes.c_int64, ctypes.c_double)
        vp = ctypes.c_void_p
        L.oracle_rng_block.argtypes = [u64, u32, u32, u32, u32, u32, vp]
        L.oracle_rng_block.restype = None
        L.oracle_philox_raw.argtypes = [vp, vp, vp]
        L.oracle_philox_raw.restype = None
        L.oracle_perm.argtypes = [i32, u64, u32, u32, u32, u32, vp]
        L.oracle_perm.restype = None
        L.oracle_fold_split.argtypes = [i64, i32, u64, vp, vp]
        L.oracle_fold_split.restype = ctypes.c_int
        L.oracle_epoch_order.argtypes = [i64, i32, u64, i32, i32, i32, vp]
        L.oracle_epoch_order.restype = ctypes.c_int
        L.oracle_expf.argtypes = [ctypes.c_float]
        L.oracle_expf.restype = ctypes.c_float
        L.oracle_expf_array.argtypes = [vp, i64, vp]
        L.oracle_expf_array.restype = None
        L.oracle_rng_blocks.argtypes = [u64, vp, i64, vp]
        L.oracle_rng_blocks.restype = None
        L.oracle_param_count.argtypes = [i32, i32, i32]
        L.oracle_param_count.restype = i64
        L.oracle_init_params.argtypes = [i32, i32, i32, u64, i32, i32, vp]
        L.oracle_init_params.restype = None
        L.oracle_loss_grad.argtypes = [i32, i32, i32, i32, i32, f64, vp, vp, vp, i32, vp]
        L.oracle_loss_grad.restype = f64
        L.oracle_adam_steps.argtypes = [i32, i64, i32, f64, f64, f64, f64, vp, vp, vp, vp]
        L.oracle_adam_steps.restype = None
        L.oracle_mlp_cv_fits.argtypes = [i32, vp, vp, i64, i32, i32, i32, vp, i32, u64, i32, vp, vp,
                                         i32, i32, i32, vp, vp, vp]
        L.oracle_mlp_cv_fits.restype = ctypes.c_int
        L.oracle_mlp_cv_eval.argtypes = [i32, vp, vp, i64, i32, i32, i32, vp, i32, u64, i32, i32, i32,
                                         vp, vp, vp]
        L.oracle_mlp_cv_eval.restype = ctypes.c_int
        L.oracle_mlp_cv_fits_ex.argtypes = L.oracle_mlp_cv_fits.argtypes + [i32, i32]
        L.oracle_mlp_cv_fits_ex.restype = ctypes.c_int
        L.oracle_mlp_cv_eval_ex.argtypes = L.oracle_mlp_cv_eval.argtypes + [i32, i32]
        L.oracle_mlp_cv_eval_ex.restype = ctypes.c_int
        L.oracle_sgd_steps.argtypes = [i32, i64, i32, f64, f64, vp, vp, vp]
        L.oracle_sgd_steps.restype = None
        L.oracle_mlp_holdout_eval.argtypes = [i32, vp, vp, i64, vp, vp, i64, i32, i32, vp, i32, u64, i32, i32, i32,
                                              i32, vp, vp]
        L.oracle_mlp_holdout_eval.restype = ctypes.c_int
        L.oracle_holdout_order.argtypes = [i64, u64, i32, i32, vp]
        L.oracle_holdout_order.restype = ctypes.c_int
        L.oracle_num_procs.restype = ctypes.c_int
        L.oracle_tf32_round.argtypes = [ctypes.c_float]
        L.oracle_tf32_round.restype = ctypes.c_float
        L.oracle_tf32_split.argtypes = [ctypes.c_float, vp, vp]
        L.oracle_tf32_split.restype = None
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def rng_block(seed, stream, a, b, c, blk):
    out = np.zeros(4, np.uint32)
    lib().oracle_rng_block(seed, stream, a, b, c, blk, _p(out))
    return out


def philox_raw(ctr, key):
    ctr = np.asarray(ctr, np.uint32)
    key = np.asarray(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().oracle_philox_raw(_p(ctr), _p(key), _p(out))
    return out


def perm(N, seed, stream, a=0, b=0, c=0):
    out = np.zeros(N, np.int32)
    lib().oracle_perm(N, seed, stream, a, b, c, _p(out))
    return out


def fold_split(n, K, seed):
    """Returns (pi, fold_of_row)."""
    pi = np.zeros(n, np.int32)
    fo = np.full(n, -1, np.int32)
    if lib().oracle_fold_split(n, K, seed, _p(pi), _p(fo)) != 0:
        raise ValueError("invalid fold split arguments")
    return pi, fo


def epoch_order(n, K, seed, config, fold, epoch):
    out = np.zeros(n, np.int32)
    m = lib().oracle_epoch_order(n, K, seed, config, fold, epoch, _p(out))
    if m < 0:
        raise ValueError("invalid arguments")
    return out[:m].copy()


def expf(x):
    return float(lib().oracle_expf(float(x)))


def expf_array(x):
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty_like(x)
    lib().oracle_expf_array(_p(x), x.size, _p(out))
    return out


def rng_blocks(seed, counters):
    """counters [count, 5] = (stream, a, b, c, blk) -> words [count, 4]."""
    counters = np.ascontiguousarray(counters, np.uint32).reshape(-1, 5)
    out = np.empty((counters.shape[0], 4), np.uint32)
    lib().oracle_rng_blocks(seed, _p(counters), counters.shape[0], _p(out))
    return out


def param_count(d, H, C):
    return int(lib().oracle_param_count(d, H, C))


def init_params(d, H, C, seed, config, fold):
    th = np.zeros(param_count(d, H, C), np.float64)
    lib().oracle_init_params(d, H, C, seed, config, fold, _p(th))
    return th


def loss_grad(mode, d, H, C, task, alpha, theta, xb, yb):
    theta = np.ascontiguousarray(theta, np.float64)
    xb = np.ascontiguousarray(xb, np.float64)
    yb = np.ascontiguousarray(yb, np.float64)
    g = np.zeros_like(theta)
    loss = lib().oracle_loss_grad(mode, d, H, C, task, float(alpha), _p(theta), _p(xb), _p(yb),
                                  xb.shape[0], _p(g))
    return loss, g


def adam_steps(mode, theta, m, v, grads, lr, beta1, beta2, eps):
    theta = np.array(theta, np.float64)
    m = np.array(m, np.float64)
    v = np.array(v, np.float64)
    grads = np.ascontiguousarray(grads, np.float64).reshape(-1, theta.size)
    lib().oracle_adam_steps(mode, theta.size, grads.shape[0], lr, beta1, beta2, eps, _p(theta), _p(m),
                            _p(v), _p(grads))
    return theta, m, v


def sgd_steps(mode, theta, vel, grads, lr, momentum):
    """n momentum-SGD updates with the given gradients [n, P]; returns (theta, velocity)."""
    theta = np.array(theta, np.float64)
    vel = np.array(vel, np.float64)
    grads = np.ascontiguousarray(grads, np.float64).reshape(-1, theta.size)
    lib().oracle_sgd_steps(mode, theta.size, grads.shape[0], lr, momentum, _p(theta), _p(vel), _p(grads))
    return theta, vel


def _prep(X, y, configs):
    X = np.ascontiguousarray(X, np.float32)
    y = np.ascontiguousarray(y, np.float32)
    configs = np.ascontiguousarray(configs)
    assert configs.dtype.itemsize == 32
    return X, y, configs


def cv_fits(X, y, task, n_folds, configs, seed, fit_config, fit_fold, mode=MODE_F32, n_classes=0,
            trace_steps=0, n_threads=0, want_theta=False, solver=SOLVER_ADAM, metric=METRIC_DEFAULT):
    """Run the listed (config, fold) fits.  Returns dict(scores, trace, theta).

    solver: SOLVER_ADAM or SOLVER_SGD (Nesterov momentum = the configuration's beta1);
    metric: METRIC_DEFAULT (accuracy / -MSE) or METRIC_ALT (-NLL / -MAE)."""
    X, y, configs = _prep(X, y, configs)
    n, d = X.shape
    fc = np.ascontiguousarray(fit_config, np.int32)
    ff = np.ascontiguousarray(fit_fold, np.int32)
    scores = np.zeros(fc.size, np.float64)
    trace = np.zeros((fc.size, trace_steps), np.float64) if trace_steps else None
    theta = None
    if want_theta:
        C = 1 if task == 1 else (n_classes or int(y.max()) + 1)
        theta = np.zeros(param_count(d, int(configs["hidden"][fc[-1]]), C), np.float64)
    rc = lib().oracle_mlp_cv_fits_ex(mode, _p(X), _p(y), n, d, task, n_folds, _p(configs), configs.size, seed,
                                     n_classes, _p(fc), _p(ff), fc.size, trace_steps, n_threads, _p(scores),
                                     _p(trace), _p(theta), solver, metric)
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return dict(scores=scores, trace=trace, theta=theta)


def cv_eval(X, y, task, n_folds, configs, seed, mode=MODE_F32, n_classes=0, trace_steps=0, n_threads=0,
            solver=SOLVER_ADAM, metric=METRIC_DEFAULT):
    """scores = evaluate(params_list).  Returns dict(scores, fold_scores, trace)."""
    X, y, configs = _prep(X, y, configs)
    n, d = X.shape
    nc = configs.size
    scores = np.zeros(nc, np.float64)
    fold_scores = np.zeros((nc, n_folds), np.float64)
    trace = np.zeros((nc * n_folds, trace_steps), np.float64) if trace_steps else None
    rc = lib().oracle_mlp_cv_eval_ex(mode, _p(X), _p(y), n, d, task, n_folds, _p(configs), nc, seed, n_classes,
                                     trace_steps, n_threads, _p(scores), _p(fold_scores), _p(trace), solver, metric)
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return dict(scores=scores, fold_scores=fold_scores, trace=trace)


HOLDOUT_FOLD_KEY = 0xFFFF


def holdout_eval(X, y, Xtest, ytest, task, configs, seed, mode=MODE_F32, n_classes=0, n_threads=0,
                 solver=SOLVER_ADAM, metric=METRIC_DEFAULT, want_theta=False):
    """One fit per configuration on all rows of (X, y), scored on (Xtest, ytest).
    Returns dict(scores, theta) (theta: parameters of the last configuration's fit)."""
    X, y, configs = _prep(X, y, configs)
    Xtest = np.ascontiguousarray(Xtest, np.float32)
    ytest = np.ascontiguousarray(ytest, np.float32)
    n, d = X.shape
    scores = np.zeros(configs.size, np.float64)
    theta = None
    if want_theta:
        C = 1 if task == 1 else (n_classes or int(max(y.max(), ytest.max())) + 1)
        theta = np.zeros(param_count(d, int(configs["hidden"][-1]), C), np.float64)
    rc = lib().oracle_mlp_holdout_eval(mode, _p(X), _p(y), n, _p(Xtest), _p(ytest), Xtest.shape[0], d, task,
                                       _p(configs), configs.size, seed, n_classes, solver, metric, n_threads,
                                       _p(scores), _p(theta))
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return dict(scores=scores, theta=theta)


def holdout_order(n, seed, config, epoch):
    out = np.zeros(n, np.int32)
    assert lib().oracle_holdout_order(n, seed, config, epoch, _p(out)) == 0
    return out


def tf32_round(x):
    """Round-to-nearest-even of a float to the 10-bit mantissa of the TF32 operand format."""
    return float(lib().oracle_tf32_round(float(x)))


def tf32_split(x):
    """(hi, lo) with hi = tf32_round(x), lo = tf32_round(x - hi)."""
    hi, lo = ctypes.c_float(), ctypes.c_float()
    lib().oracle_tf32_split(float(x), ctypes.byref(hi), ctypes.byref(lo))
    return hi.value, lo.value


def num_procs():
    return int(lib().oracle_num_procs())
