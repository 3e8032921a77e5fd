/* bbo_mlp_cv.h -- C ABI of the fused MLP-Adam cross-validation library (CUDA, sm_100a).
 *
 * The library is the `evaluate(params_list) -> scores` call of the suggest-observe loop
 * (paper, Algorithm 1): for every suggested hyperparameter configuration it returns the
 * k-fold cross-validation score of one model / dataset / metric triple, which is the function
 * the optimizers of the paper see (sec. 2), for the model the paper's Table 1 calls MLP-adam,
 * with the metrics acc and mse of the same table, five folds in the paper's runs (sec. 6.3:
 * 2.7 M trainings for 541,440 evaluations).  Function evaluation is what the paper moves to the GPU because it
 * dominates run time (sec. 1, sec. 5, sec. 6.3).
 *
 * Model and training rule (the paper names the model, not its formulas; these are the
 * readings this library fixes): one hidden ReLU layer of width `hidden`; softmax
 * cross-entropy averaged over the minibatch (classification) or half the mean squared error
 * (regression); L2 penalty alpha/(2*batch) on both weight matrices; Adam with step size
 * lr*sqrt(1-beta2^t)/(1-beta1^t) and update m/(sqrt(v)+eps); Glorot-uniform initial
 * weights and biases; shuffled, non-stratified k-fold split shared by all configurations;
 * a fresh minibatch permutation every epoch, last short batch kept.  All random choices come
 * from Philox-4x32-10 keyed by `seed` and indexed by (configuration index, fold, epoch or
 * layer, element), so a score depends only on its own configuration, its index in the list
 * and the seed -- never on the other entries, the grid or the scheduling.
 *
 * Variants selected per handle (bbo_mlp_cv_options): the MLP-sgd update rule and the nll / mae
 * metrics of the paper's Table 1; bbo_mlp_cv_eval_holdout gives the generalisation score of
 * sec. 6.2 (train on all rows, score a held-out matrix).
 *
 * No C++ types, no exceptions and no printing cross this boundary.  Every function returns
 * 0 on success or a negative bbo_status.  All floating point is IEEE binary32 unless noted.
 */
#ifndef BBO_MLP_CV_H_
#define BBO_MLP_CV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bbo_mlp_cv bbo_mlp_cv; /* opaque handle */

/* One suggested configuration (an element of Algorithm 1's params_list).  POD, 32 bytes. */
typedef struct {
  int32_t hidden;     /* H >= 1, at most the cap reported by bbo_mlp_cv_query_caps        */
  int32_t batch_size; /* B >= 1; the effective size is min(B, training rows of the fold)   */
  int32_t epochs;     /* E in [0, 2^28); 0 scores the initial weights                      */
  float alpha;        /* L2 strength >= 0                                                   */
  float lr;           /* Adam learning rate >= 0                                            */
  float beta1, beta2; /* in [0, 1)                                                          */
  float eps;          /* > 0                                                                */
} bbo_mlp_config;

typedef enum { BBO_TASK_CLASSIFICATION = 0, BBO_TASK_REGRESSION = 1 } bbo_task;

/* Update rule of every fit of a handle (paper, Table 1 lists MLP-adam and MLP-sgd).
 * BBO_SOLVER_SGD is stochastic gradient descent with Nesterov momentum and a constant
 * learning rate: velocity = momentum*velocity - lr*g; theta += momentum*velocity - lr*g (the
 * second expression with the new velocity; lr*g rounded once, each expression one fused
 * multiply-add).  The momentum is the configuration's beta1; beta2 and eps are ignored.     */
typedef enum { BBO_SOLVER_ADAM = 0, BBO_SOLVER_SGD = 1 } bbo_solver;

/* Held-out score (paper, Table 1: metrics acc, nll for classifiers; mse, mae for regressors).
 * BBO_METRIC_DEFAULT: accuracy, or minus the mean squared error.  BBO_METRIC_ALT: minus the
 * mean negative log-likelihood of the true class under the softmax, or minus the mean absolute
 * error (row sums in ascending row order; NaN maps to -inf).  Always "higher is better".    */
typedef enum { BBO_METRIC_DEFAULT = 0, BBO_METRIC_ALT = 1 } bbo_metric;

/* Arithmetic of the two large contractions (paper sec. 5 only says the MLP is "GPU-optimized").
 * BBO_VARIANT_FP32: binary32 fused multiply-adds on the CUDA cores in one fixed order; the only
 * variant that is built, because the score tolerance (1e-3 on accuracies whose quantum is one
 * held-out row) needs identical predictions after tens of thousands of optimizer steps.
 * BBO_VARIANT_TF32 names the tensor-core variant (TF32 operands, with or without a high/low
 * operand split); the CPU checker's experiment modes show that neither keeps 99 % of the fold
 * scores within the tolerance, so bbo_mlp_cv_create answers BBO_ERR_UNSUPPORTED for it.       */
typedef enum { BBO_VARIANT_FP32 = 0, BBO_VARIANT_TF32 = 1 } bbo_variant;

typedef enum {
  BBO_OK = 0,
  BBO_ERR_INVALID_ARG = -1, /* NULL pointer, bad size, hyperparameter or label out of range */
  BBO_ERR_UNSUPPORTED = -2, /* shape above the kernel caps, or not an sm_100 device         */
  BBO_ERR_CUDA = -3,        /* a CUDA runtime call failed (see bbo_mlp_cv_last_cuda_error)  */
  BBO_ERR_TIMEOUT = -4,     /* a bounded device-side wait gave up                           */
  BBO_ERR_OOM = -5,         /* scratch allocation failed                                    */
  BBO_ERR_TOO_LARGE = -6    /* problem exceeds the fixed scratch of bbo_mlp_cv_eval_static  */
} bbo_status;

/* Create-time options; a zeroed struct selects the defaults. */
typedef struct {
  int32_t device;      /* CUDA ordinal; -1 = the calling thread's current device            */
  void* stream;        /* cudaStream_t borrowed from the caller; NULL = the default stream  */
  int32_t n_classes;   /* classification: 0 = 1 + max(y) found on the device                */
  int32_t trace_steps; /* >0: record the minibatch training loss of the first N optimizer
                          steps of every fit (debug / parity; slows the kernel)             */
  int32_t keep_theta;  /* 1: keep the final parameters of the LAST fit of the list, i.e.
                          (configuration n_configs-1, fold n_folds-1), for
                          bbo_mlp_cv_debug_theta                                            */
  int32_t config_index_base; /* added to each configuration's position in the list when keying
                          its random streams: a caller that splits one params_list over several
                          handles (e.g. one per GPU) passes the position of its first entry and
                          gets the scores the unsplit call would give                          */
  int32_t solver;      /* a bbo_solver; 0 = Adam                                             */
  int32_t metric;      /* a bbo_metric; 0 = accuracy / minus mean squared error               */
  int32_t variant;     /* a bbo_variant; 0 = FP32 CUDA cores (the only one built)             */
} bbo_mlp_cv_options;

/* Creates a handle bound to one device and one stream.  `opt` may be NULL (defaults).
 * The handle owns its scratch buffers (grown on demand, freed by destroy).               */
int bbo_mlp_cv_create(const bbo_mlp_cv_options* opt, bbo_mlp_cv** out);

/* scores = evaluate(params_list) (paper, Algorithm 1; sec. 2).
 *   X          DEVICE, row-major [n*d] float, 4-byte aligned; read only
 *   y          DEVICE [n] float: class ids 0..C-1 stored exactly, or regression targets
 *   n, d       rows and features; task  a bbo_task; n_folds  2 <= K <= n
 *   configs    HOST [n_configs]; copied during the call
 *   seed       keys the fold split, every initialisation and every minibatch order
 *   out_scores DEVICE [n_configs] float: mean over folds (ascending fold, float sum, then
 *              one division) of held-out accuracy, or of minus the held-out mean squared
 *              error (higher is better; a NaN error maps to -inf)
 * Work is enqueued on the handle's stream, which is synchronised before returning, so the
 * status reflects the device's and out_scores is ready.  The caller keeps ownership of all
 * four buffers; none is retained.  On error out_scores is unspecified.  One call at a time
 * per handle; distinct handles are independent.                                           */
int bbo_mlp_cv_eval(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d,
                    int32_t task, int32_t n_folds, const bbo_mlp_config* configs,
                    int32_t n_configs, uint64_t seed, float* out_scores);

/* As bbo_mlp_cv_eval, with an explicit key per configuration for its random streams instead of
 * its position in the list (paper sec. 5 deals the jobs to the GPUs in round-robin order: a
 * caller that splits one params_list unevenly, e.g. balanced by cost, passes each entry's
 * position in the unsplit list and gets exactly the scores of the unsplit call).
 *   config_keys  HOST [n_configs], each in [0, 2^28); copied during the call
 * The handle's config_index_base is ignored by this call.                                   */
int bbo_mlp_cv_eval_keyed(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d,
                          int32_t task, int32_t n_folds, const bbo_mlp_config* configs,
                          const int32_t* config_keys, int32_t n_configs, uint64_t seed,
                          float* out_scores);

/* Hold-out ("generalisation") scores of the same configurations (paper, sec. 6.2: the data
 * are split into the part the optimizers see through cross-validation and a part held out to
 * measure generalisation).  One fit per configuration: trained on all n rows of (X, y), in the
 * order of the fold permutation of `seed`, with the minibatch and initialisation streams keyed
 * by fold index 65535, then scored on the n_test rows of (Xtest, ytest) in their own order.
 *   X, y, Xtest, ytest  DEVICE, layouts as in bbo_mlp_cv_eval; n_test in [1, row cap]
 *   out_scores          DEVICE [n_configs]: the handle's metric on the test rows
 * The class count covers the labels of both parts.  Ownership, synchrony and errors as in
 * bbo_mlp_cv_eval; bbo_mlp_cv_fold_scores then returns one value per configuration.        */
int bbo_mlp_cv_eval_holdout(bbo_mlp_cv* h, const float* X, const float* y, int64_t n,
                            const float* Xtest, const float* ytest, int64_t n_test, int32_t d,
                            int32_t task, const bbo_mlp_config* configs, int32_t n_configs,
                            uint64_t seed, float* out_scores);

/* As bbo_mlp_cv_eval, with X, y and out_scores in HOST memory: copies them to device
 * scratch owned by the handle, evaluates, copies the scores back.                         */
int bbo_mlp_cv_eval_host(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d,
                         int32_t task, int32_t n_folds, const bbo_mlp_config* configs,
                         int32_t n_configs, uint64_t seed, float* out_scores);

int bbo_mlp_cv_destroy(bbo_mlp_cv* h);

/* Results of the last eval kept by the handle (HOST output buffers).
 *   fold_scores: [n_configs*n_folds], configuration-major
 *   loss_trace:  [n_configs*n_folds*trace_steps], NaN where a fit had fewer steps
 *   theta:       W1[d][H] row-major, b1[H], W2[H][C] row-major, b2[C] of the kept fit;
 *                `count` must equal that parameter count                                  */
int bbo_mlp_cv_fold_scores(bbo_mlp_cv* h, float* host_out, int64_t count);
int bbo_mlp_cv_loss_trace(bbo_mlp_cv* h, float* host_out, int64_t count);
int bbo_mlp_cv_debug_theta(bbo_mlp_cv* h, float* host_out, int64_t count);

/* Runs the DEVICE index code and copies the result back (parity of the fold split and the
 * minibatch order).  host_fold_of_row[n]: fold in which each row is held out.
 * host_order[n - size of that fold]: dataset row visited i-th in `epoch` of fit
 * (config, fold); minibatch s of size B is host_order[s*B .. s*B+B).  Either may be NULL. */
int bbo_mlp_cv_debug_indices(bbo_mlp_cv* h, int64_t n, int32_t n_folds, uint64_t seed,
                             int32_t config, int32_t fold, int32_t epoch,
                             int32_t* host_fold_of_row, int32_t* host_order);

/* Device-side Philox block and the float exponential used by the softmax, for bit-exact
 * comparison with another implementation.  counters: HOST [count*5] words
 * (stream, a, b, c, blk); out: HOST [count*4].  x, out: HOST [count].                     */
int bbo_mlp_cv_debug_rng(bbo_mlp_cv* h, uint64_t seed, const uint32_t* counters, int64_t count,
                         uint32_t* out);
int bbo_mlp_cv_debug_exp(bbo_mlp_cv* h, const float* x, int64_t count, float* out);

/* The Adam update needs one IEEE square root and one IEEE division per parameter per step,
 * the softmax one IEEE division per class and row; the kernels use branch-free FMA-corrected
 * versions inside a safe exponent range and the IEEE routines outside it.  This export
 * compares the two on the device.  mode 0: square root of the `count` float bit patterns
 * starting at `first`; mode 1: m / (sqrt(v) + eps) on `count` pseudo-random operand triples
 * keyed by `seed`; mode 3: the same quotient with denormal or tiny m, so that most results
 * are denormal; mode 2: softmax quotients exp(-t) / s, t in [0, 90), s in [1, 16], on
 * `count` pseudo-random pairs.  host_out4: HOST [4] = number of
 * bit-level disagreements, number of cases taken by the fast path, and (for diagnosis) the
 * operand bits of one disagreement.                                                       */
int bbo_mlp_cv_debug_fast_math(bbo_mlp_cv* h, int32_t mode, uint64_t seed, uint64_t first,
                               uint64_t count, uint64_t* host_out4);

/* Measures the FP32 fused-multiply-add rate this device sustains from registers (no memory
 * traffic): every SM runs `threads_per_sm` threads doing `iters` rounds of 16 independent
 * FMAs.  *tflops receives 2 * FMAs / time.  It is the roofline ceiling the fit kernel is
 * compared with, measured at the clock the device actually holds.                          */
int bbo_mlp_cv_debug_ffma_peak(bbo_mlp_cv* h, int32_t threads_per_sm, int32_t iters, float* tflops);

/* Largest shapes one call accepts on this device: rows, features, hidden width for the
 * given (d, n_classes) pair, and classes.  The hidden-width and feature caps are those of a
 * 1797-row, 5-fold problem; they shrink for longer training folds (the per-epoch sort scratch
 * grows with the fold).  Any output pointer may be NULL.                                  */
int bbo_mlp_cv_query_caps(bbo_mlp_cv* h, int32_t d, int32_t n_classes, int32_t* max_n,
                          int32_t* max_d, int32_t* max_hidden, int32_t* max_classes);

/* Device time (CUDA events on the handle's stream) of the last eval in milliseconds:
 * total_ms from before the first kernel (row padding / fold permutation) to after the fold
 * mean, fit_ms around the fit kernel alone; and the number of kernels the eval launched.
 * Any pointer may be NULL.                                                                */
int bbo_mlp_cv_last_timing(bbo_mlp_cv* h, float* total_ms, float* fit_ms, int32_t* n_launches);

/* Allocation-free evaluation.  (The paper has no counterpart to this call; it exists for
 * the library's users.)  Same result as bbo_mlp_cv_eval, for callers that must not allocate
 * device memory while they run: code inside a memory-pool or arena framework that owns the
 * whole device heap, real-time or latency-bound loops where cudaMalloc's implicit device
 * synchronisation and unbounded latency are not acceptable, and processes that have already
 * handed all free memory to another component.  It needs no handle, and it calls neither
 * cudaMalloc nor cudaFree nor any allocating library routine (what the driver itself does when
 * a kernel is launched for the first time is described below).
 *
 * All working memory (fold permutation, device copy of the configurations, fit list,
 * per-fold scores, work counter, padded copy of X) lives in ONE fixed array of
 * BBO_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds those bytes until the process exits, used or not.  Hence the limits, checked
 * before anything is enqueued and reported as BBO_ERR_TOO_LARGE:
 *     n <= BBO_STATIC_MAX_ROWS,  n * roundup8(d) <= BBO_STATIC_MAX_X_FLOATS,
 *     n_configs <= BBO_STATIC_MAX_CONFIGS,  n_configs * n_folds <= BBO_STATIC_MAX_FITS.
 * Shapes above the kernel caps are BBO_ERR_UNSUPPORTED as in bbo_mlp_cv_eval.
 *
 *   stream     cudaStream_t of the CURRENT device (NULL = default stream); work is enqueued
 *              there and the stream is synchronised before returning
 *   X, y, out_scores  DEVICE buffers of the current device, as in bbo_mlp_cv_eval
 *   n_classes  classification: 0 = 1 + max(y) found on the device; ignored for regression
 *   configs    HOST [n_configs]
 *
 * The call is synchronous: it synchronises the stream twice (after the label scan and at the
 * end) and copies from pageable host memory, so it cannot run inside a stream capture.  The
 * first call on each device also looks up the array's device address and the device's limits
 * (a one-off set-up, cached per device), and the first launch of each kernel instance lets the
 * driver load that kernel's code, which may take device memory inside the driver: a warm-up
 * call per data shape, made while allocation is still allowed, gets both out of the way.  The
 * array is shared by every call in the process and keeps the previous call's contents; the
 * call clears what has to start from zero.  Two calls that overlap on the same GPU (different
 * streams or threads) would race on it: run them one after another.
 * bbo_mlp_cv_static_last_cuda_error returns the text of the calling thread's last CUDA error
 * from this entry point ("" if none).                                                        */
#define BBO_STATIC_MAX_ROWS 4096
#define BBO_STATIC_MAX_X_FLOATS 262144
#define BBO_STATIC_MAX_CONFIGS 4096
#define BBO_STATIC_MAX_FITS 16384
#define BBO_STATIC_SCRATCH_BYTES (256 + 4 * BBO_STATIC_MAX_ROWS + 32 * BBO_STATIC_MAX_CONFIGS + \
                                  12 * BBO_STATIC_MAX_FITS + 4 * BBO_STATIC_MAX_X_FLOATS)
int bbo_mlp_cv_eval_static(void* stream, const float* X, const float* y, int64_t n, int32_t d,
                           int32_t task, int32_t n_folds, int32_t n_classes,
                           const bbo_mlp_config* configs, int32_t n_configs, uint64_t seed,
                           float* out_scores);

const char* bbo_mlp_cv_static_last_cuda_error(void);

const char* bbo_mlp_cv_strerror(int code);
/* Text of the last CUDA error seen by this handle ("" if none).  Valid until the next call. */
const char* bbo_mlp_cv_last_cuda_error(bbo_mlp_cv* h);

#ifdef __cplusplus
}
#endif
#endif /* BBO_MLP_CV_H_ */
