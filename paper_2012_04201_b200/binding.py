"""ctypes binding over ``libbbo_mlp_cv.so``: argument marshalling only.

Every step of the evaluation runs in the CUDA library; nothing here computes.  The
functions carry the C names (``bbo_mlp_cv_create`` ... ``bbo_mlp_cv_destroy``); the
:class:`MlpCv` wrapper adds tensor/array conversion.  PyTorch supplies device memory and
streams.  If the library is missing it is built with nvcc; if that is impossible the
import of the library raises -- there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build
from .workloads import CONFIG_DTYPE

BBO_OK = 0
BBO_ERR_INVALID_ARG = -1
BBO_ERR_UNSUPPORTED = -2
BBO_ERR_CUDA = -3
BBO_ERR_TIMEOUT = -4
BBO_ERR_OOM = -5
BBO_ERR_TOO_LARGE = -6

TASK_CLASSIFICATION = 0
TASK_REGRESSION = 1
SOLVER_ADAM, SOLVER_SGD = 0, 1
METRIC_DEFAULT, METRIC_ALT = 0, 1
VARIANT_FP32, VARIANT_TF32 = 0, 1

EXPORTS = [
    "bbo_mlp_cv_create", "bbo_mlp_cv_eval", "bbo_mlp_cv_eval_host", "bbo_mlp_cv_eval_holdout", "bbo_mlp_cv_destroy",
    "bbo_mlp_cv_eval_keyed", "bbo_mlp_cv_static_last_cuda_error",
    "bbo_mlp_cv_fold_scores", "bbo_mlp_cv_loss_trace", "bbo_mlp_cv_debug_theta",
    "bbo_mlp_cv_debug_indices", "bbo_mlp_cv_debug_rng", "bbo_mlp_cv_debug_exp",
    "bbo_mlp_cv_query_caps", "bbo_mlp_cv_last_timing", "bbo_mlp_cv_strerror",
    "bbo_mlp_cv_last_cuda_error", "bbo_mlp_cv_eval_static", "bbo_mlp_cv_debug_fast_math", "bbo_mlp_cv_debug_ffma_peak",
]


class Options(ctypes.Structure):
    _fields_ = [("device", ctypes.c_int32), ("stream", ctypes.c_void_p), ("n_classes", ctypes.c_int32),
                ("trace_steps", ctypes.c_int32), ("keep_theta", ctypes.c_int32),
                ("config_index_base", ctypes.c_int32), ("solver", ctypes.c_int32), ("metric", ctypes.c_int32),
                ("variant", ctypes.c_int32)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load():
    """Loads (building first if needed) the CUDA library.  Raises if it cannot."""
    global _lib
    if _lib is not None:
        return _lib
    if _build.needs_build():
        try:
            _build.build()
        except Exception as exc:  # no nvcc and no prebuilt library: fail loudly
            if not os.path.exists(_build.LIB):
                raise RuntimeError(
                    "libbbo_mlp_cv.so is missing and could not be built; run "
                    "`python -m paper_2012_04201_b200.build` on a machine with nvcc") from exc
    L = ctypes.CDLL(_build.LIB)
    i32, i64, u64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p
    L.bbo_mlp_cv_create.argtypes = [ctypes.POINTER(Options), ctypes.POINTER(vp)]
    L.bbo_mlp_cv_eval.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp, i32, u64, vp]
    L.bbo_mlp_cv_eval_host.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp, i32, u64, vp]
    L.bbo_mlp_cv_eval_keyed.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp, vp, i32, u64, vp]
    L.bbo_mlp_cv_static_last_cuda_error.argtypes = []
    L.bbo_mlp_cv_static_last_cuda_error.restype = ctypes.c_char_p
    L.bbo_mlp_cv_eval_holdout.argtypes = [vp, vp, vp, i64, vp, vp, i64, i32, i32, vp, i32, u64, vp]
    L.bbo_mlp_cv_destroy.argtypes = [vp]
    L.bbo_mlp_cv_eval_static.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, i32, u64, vp]
    L.bbo_mlp_cv_fold_scores.argtypes = [vp, vp, i64]
    L.bbo_mlp_cv_loss_trace.argtypes = [vp, vp, i64]
    L.bbo_mlp_cv_debug_theta.argtypes = [vp, vp, i64]
    L.bbo_mlp_cv_debug_indices.argtypes = [vp, i64, i32, u64, i32, i32, i32, vp, vp]
    L.bbo_mlp_cv_debug_rng.argtypes = [vp, u64, vp, i64, vp]
    L.bbo_mlp_cv_debug_exp.argtypes = [vp, vp, i64, vp]
    L.bbo_mlp_cv_debug_fast_math.argtypes = [vp, i32, u64, u64, u64, vp]
    L.bbo_mlp_cv_debug_ffma_peak.argtypes = [vp, i32, i32, vp]
    L.bbo_mlp_cv_query_caps.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.bbo_mlp_cv_last_timing.argtypes = [vp, vp, vp, vp]
    L.bbo_mlp_cv_strerror.argtypes = [ctypes.c_int]
    L.bbo_mlp_cv_strerror.restype = ctypes.c_char_p
    L.bbo_mlp_cv_last_cuda_error.argtypes = [vp]
    L.bbo_mlp_cv_last_cuda_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("bbo_mlp_cv_strerror", "bbo_mlp_cv_last_cuda_error", "bbo_mlp_cv_static_last_cuda_error"):
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


class BboError(RuntimeError):
    def __init__(self, code, detail=""):
        self.code = code
        msg = load().bbo_mlp_cv_strerror(code).decode()
        super().__init__(f"bbo_mlp_cv: {msg} ({code})" + (f": {detail}" if detail else ""))


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


# ---- functions with the C names -------------------------------------------------------
def bbo_mlp_cv_create(device=-1, stream=0, n_classes=0, trace_steps=0, keep_theta=0, config_index_base=0,
                      solver=SOLVER_ADAM, metric=METRIC_DEFAULT, variant=VARIANT_FP32):
    opt = Options(device=device, stream=stream or None, n_classes=n_classes, trace_steps=trace_steps,
                  keep_theta=int(keep_theta), config_index_base=int(config_index_base), solver=int(solver),
                  metric=int(metric), variant=int(variant))
    h = ctypes.c_void_p()
    rc = load().bbo_mlp_cv_create(ctypes.byref(opt), ctypes.byref(h))
    if rc != BBO_OK:
        raise BboError(rc)
    return h


def bbo_mlp_cv_eval(h, X_ptr, y_ptr, n, d, task, n_folds, configs, seed, out_ptr):
    """Device pointers (ints) for X, y, out; ``configs`` a CONFIG_DTYPE array.  Returns rc."""
    configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
    return load().bbo_mlp_cv_eval(h, X_ptr, y_ptr, n, d, task, n_folds, _np_ptr(configs), configs.size,
                                  seed, out_ptr)


def bbo_mlp_cv_eval_keyed(h, X_ptr, y_ptr, n, d, task, n_folds, configs, config_keys, seed, out_ptr):
    """As bbo_mlp_cv_eval with one random-stream key per configuration (int32 array)."""
    configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
    keys = np.ascontiguousarray(config_keys, dtype=np.int32)
    assert keys.size == configs.size
    return load().bbo_mlp_cv_eval_keyed(h, X_ptr, y_ptr, n, d, task, n_folds, _np_ptr(configs), _np_ptr(keys),
                                        configs.size, seed, out_ptr)


def bbo_mlp_cv_eval_host(h, X, y, task, n_folds, configs, seed, out):
    configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
    return load().bbo_mlp_cv_eval_host(h, _np_ptr(X), _np_ptr(y), X.shape[0], X.shape[1], task, n_folds,
                                       _np_ptr(configs), configs.size, seed, _np_ptr(out))


def bbo_mlp_cv_destroy(h):
    return load().bbo_mlp_cv_destroy(h)


def bbo_mlp_cv_eval_static(stream_ptr, X_ptr, y_ptr, n, d, task, n_folds, n_classes, configs, seed, out_ptr):
    """Allocation-free evaluation on the current device (no handle).  Device pointers (ints)
    for X, y, out; ``configs`` a CONFIG_DTYPE array.  All device scratch comes from a fixed
    array inside the library, so the call never asks the driver for memory; problems above
    the documented limits return BBO_ERR_TOO_LARGE.  Returns the status code."""
    configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
    return load().bbo_mlp_cv_eval_static(stream_ptr or None, X_ptr, y_ptr, n, d, task, n_folds, n_classes,
                                         _np_ptr(configs), configs.size, seed, out_ptr)


# ---- convenience wrapper ---------------------------------------------------------------
class MlpCv:
    """One handle = one device, one stream, one call in flight."""

    def __init__(self, device=None, stream=None, n_classes=0, trace_steps=0, keep_theta=False, config_index_base=0,
                 solver=SOLVER_ADAM, metric=METRIC_DEFAULT, variant=VARIANT_FP32):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("bbo_mlp_cv needs a CUDA device (there is no CPU path)")
        self._torch = torch
        self.device = torch.cuda.current_device() if device is None else int(device)
        torch.cuda.init()
        with torch.cuda.device(self.device):
            torch.zeros(1, device="cuda")  # make sure the primary context exists
        self.stream = stream
        sptr = 0 if stream is None else int(stream.cuda_stream)
        self._h = bbo_mlp_cv_create(self.device, sptr, n_classes, trace_steps, keep_theta, config_index_base,
                                    solver, metric, variant)
        self._n_configs = self._n_folds = 0
        self.trace_steps = trace_steps

    def _check(self, rc):
        if rc != BBO_OK:
            raise BboError(rc, load().bbo_mlp_cv_last_cuda_error(self._h).decode())

    def eval(self, X, y, task, n_folds, configs, seed, out=None, config_keys=None):
        """``X`` [n, d], ``y`` [n]: float32 CUDA tensors.  Returns scores [n_configs] (CUDA).
        ``config_keys``: optional int32 key per configuration for its random streams."""
        torch = self._torch
        assert X.is_cuda and y.is_cuda and X.dtype == torch.float32 and y.dtype == torch.float32
        X = X.contiguous()
        y = y.contiguous()
        configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
        if out is None:
            out = torch.empty(configs.size, dtype=torch.float32, device=X.device)
        if self.stream is not None:
            self.stream.wait_stream(torch.cuda.current_stream(X.device))
        if config_keys is None:
            rc = bbo_mlp_cv_eval(self._h, X.data_ptr(), y.data_ptr(), X.shape[0], X.shape[1], task, n_folds,
                                 configs, seed, out.data_ptr())
        else:
            rc = bbo_mlp_cv_eval_keyed(self._h, X.data_ptr(), y.data_ptr(), X.shape[0], X.shape[1], task, n_folds,
                                       configs, config_keys, seed, out.data_ptr())
        self._check(rc)
        self._n_configs, self._n_folds = configs.size, n_folds
        return out

    def eval_holdout(self, X, y, Xtest, ytest, task, configs, seed, out=None):
        """One fit per configuration on all rows of ``X``, scored on ``Xtest`` (CUDA tensors)."""
        torch = self._torch
        for t in (X, y, Xtest, ytest):
            assert t.is_cuda and t.dtype == torch.float32
        X, y, Xtest, ytest = X.contiguous(), y.contiguous(), Xtest.contiguous(), ytest.contiguous()
        assert X.shape[1] == Xtest.shape[1]
        configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
        if out is None:
            out = torch.empty(configs.size, dtype=torch.float32, device=X.device)
        if self.stream is not None:
            self.stream.wait_stream(torch.cuda.current_stream(X.device))
        rc = load().bbo_mlp_cv_eval_holdout(self._h, X.data_ptr(), y.data_ptr(), X.shape[0], Xtest.data_ptr(),
                                            ytest.data_ptr(), Xtest.shape[0], X.shape[1], task, _np_ptr(configs),
                                            configs.size, seed, out.data_ptr())
        self._check(rc)
        self._n_configs, self._n_folds = configs.size, 1
        return out

    def eval_host(self, X, y, task, n_folds, configs, seed):
        """numpy in, numpy out; the library copies to and from the device."""
        X = np.ascontiguousarray(X, np.float32)
        y = np.ascontiguousarray(y, np.float32)
        configs = np.ascontiguousarray(configs, dtype=CONFIG_DTYPE)
        out = np.empty(configs.size, np.float32)
        self._check(bbo_mlp_cv_eval_host(self._h, X, y, task, n_folds, configs, seed, out))
        self._n_configs, self._n_folds = configs.size, n_folds
        return out

    def fold_scores(self):
        out = np.empty((self._n_configs, self._n_folds), np.float32)
        self._check(load().bbo_mlp_cv_fold_scores(self._h, _np_ptr(out), out.size))
        return out

    def loss_trace(self):
        out = np.empty((self._n_configs * self._n_folds, self.trace_steps), np.float32)
        self._check(load().bbo_mlp_cv_loss_trace(self._h, _np_ptr(out), out.size))
        return out

    def debug_theta(self, count):
        out = np.empty(count, np.float32)
        self._check(load().bbo_mlp_cv_debug_theta(self._h, _np_ptr(out), count))
        return out

    def debug_indices(self, n, n_folds, seed, config, fold, epoch):
        fo = np.empty(n, np.int32)
        order = np.empty(n, np.int32)
        self._check(load().bbo_mlp_cv_debug_indices(self._h, n, n_folds, seed, config, fold, epoch,
                                                    _np_ptr(fo), _np_ptr(order)))
        n_val = n // n_folds + (1 if fold < n % n_folds else 0)
        return fo, order[: n - n_val].copy()

    def debug_rng(self, seed, counters):
        counters = np.ascontiguousarray(counters, np.uint32).reshape(-1, 5)
        out = np.empty((counters.shape[0], 4), np.uint32)
        self._check(load().bbo_mlp_cv_debug_rng(self._h, seed, _np_ptr(counters), counters.shape[0], _np_ptr(out)))
        return out

    def debug_exp(self, x):
        x = np.ascontiguousarray(x, np.float32)
        out = np.empty_like(x)
        self._check(load().bbo_mlp_cv_debug_exp(self._h, _np_ptr(x), x.size, _np_ptr(out)))
        return out

    def debug_fast_math(self, mode, seed=0, first=0, count=1):
        """(disagreements, fast-path cases, operand bits...) of the in-kernel sqrt/div check."""
        out = np.zeros(4, np.uint64)
        self._check(load().bbo_mlp_cv_debug_fast_math(self._h, mode, seed, first, count, _np_ptr(out)))
        return out

    def debug_ffma_peak(self, threads_per_sm=1024, iters=20000):
        """FP32 FMA rate (TFLOP/s) the device sustains from registers."""
        out = ctypes.c_float()
        self._check(load().bbo_mlp_cv_debug_ffma_peak(self._h, threads_per_sm, iters, ctypes.byref(out)))
        return out.value

    def query_caps(self, d, n_classes):
        v = [ctypes.c_int32() for _ in range(4)]
        self._check(load().bbo_mlp_cv_query_caps(self._h, d, n_classes, *[ctypes.byref(x) for x in v]))
        return dict(max_n=v[0].value, max_d=v[1].value, max_hidden=v[2].value, max_classes=v[3].value)

    def last_timing(self):
        """(total_ms, fit_kernel_ms, kernels launched) of the last eval, from CUDA events."""
        ms, fit, nl = ctypes.c_float(), ctypes.c_float(), ctypes.c_int32()
        self._check(load().bbo_mlp_cv_last_timing(self._h, ctypes.byref(ms), ctypes.byref(fit), ctypes.byref(nl)))
        return ms.value, fit.value, nl.value

    def close(self):
        if self._h is not None:
            bbo_mlp_cv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
