// Host side of the C ABI declared in include/bbo_mlp_cv.h: argument checks, scratch
// management, the launch sequence (label scan, row padding, fold permutation, the fit
// kernel, fold mean) and the debug exports.  scores = evaluate(params_list) of the paper's
// Algorithm 1, with the cross-validation score of sec. 2 as the evaluated function.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/bbo_mlp_cv.h"
#include "aux_kernels.cuh"
#include "fit_launch.h"

static_assert(sizeof(bbo_mlp_config) == 32, "bbo_mlp_config must be 32 bytes");
static_assert(sizeof(bbo::Config) == sizeof(bbo_mlp_config), "device mirror of bbo_mlp_config");

namespace {

using bbo::kMaxClasses;
constexpr int kAuxStreams = 32;  // buckets of different hidden width overlap on these
constexpr int kMaxRows = 16384;  // fold permutation sorts in one CTA's shared memory
constexpr int kMaxFeatures = 16384, kMaxHidden = 8192;  // beyond any shape shared memory admits; keeps the size arithmetic in int

// Device limits the launch plan needs.
struct DeviceLimits {
  int smem_optin = 0;   // largest shared memory of one CTA (static + dynamic)
  int smem_per_sm = 0;  // shared memory of one SM
  int regs_per_sm = 0;  // 32-bit registers of one SM
};

template <typename T>
struct DevBuf {
  T* p = nullptr;
  size_t cap = 0;
  cudaError_t reserve(size_t n) {
    if (n <= cap) return cudaSuccess;
    if (p) cudaFree(p);
    p = nullptr;
    cap = 0;
    cudaError_t e = cudaMalloc(&p, n * sizeof(T));
    if (e == cudaSuccess) cap = n;
    return e;
  }
  void release() {
    if (p) cudaFree(p);
    p = nullptr;
    cap = 0;
  }
};

}  // namespace

struct bbo_mlp_cv {
  int device = 0;
  cudaStream_t stream = nullptr;
  bbo_mlp_cv_options opt{};
  int sm_count = 0;
  DeviceLimits lim;
  std::string cuda_error;
  // scratch
  DevBuf<bbo::Config> configs;
  DevBuf<int2> fits;
  DevBuf<float> fold_scores, trace, theta, xpad, xpad_t, hx, hy, hscores, dbg_f;
  DevBuf<int32_t> pi, misc, dbg_i, keys;
  DevBuf<uint32_t> dbg_u;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr, evf0 = nullptr, evf1 = nullptr;
  cudaStream_t aux[kAuxStreams] = {};
  cudaEvent_t fork = nullptr, join[kAuxStreams] = {};
  // last eval
  int64_t last_fold_count = 0, last_trace_count = 0, last_theta_count = 0;
  float last_ms = 0.f, last_fit_ms = 0.f;
  int last_launches = 0;
};

namespace {

int cuda_fail(bbo_mlp_cv* h, cudaError_t e, const char* what) {
  h->cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
  return e == cudaErrorMemoryAllocation ? BBO_ERR_OOM : BBO_ERR_CUDA;
}

#define BBO_CUDA(h, call)                                       \
  do {                                                          \
    cudaError_t e_ = (call);                                    \
    if (e_ != cudaSuccess) return cuda_fail((h), e_, #call);    \
  } while (0)

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
    else prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

bool is_device_ptr(const void* p, int device) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return (at.type == cudaMemoryTypeDevice && at.device == device) || at.type == cudaMemoryTypeManaged;
}

// Launch geometry of the fits that share one padded hidden width.
struct Plan {
  int C, CS, dp, Hs, TB, NT, order_bytes, loss_cap, n_sort, per_sm;
  int extra_warps;  // pipelined schedule: warps added for the output layer (0 = plain schedule)
  int tmem_cols;
  size_t smem;
  const void* kernel;
};

// Resident CTAs per SM of a fit kernel instance (0 if it cannot launch), from the kernel's own
// registers and static shared memory, the launch's dynamic shared memory and threads, and the
// tensor-memory columns each CTA allocates (512 per SM; the occupancy query of the runtime
// does not know about those).  Also raises the instance's dynamic shared-memory limit to the
// device's opt-in maximum -- always that value, never the size of one launch: the attribute is
// global to the process, and handles on different threads share the instances.
int kernel_occupancy(const void* kernel, int threads, size_t smem, int tmem_cols, const DeviceLimits& lim) {
  cudaFuncAttributes attr;
  if (cudaFuncGetAttributes(&attr, kernel) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  const int max_dynamic = lim.smem_optin - (int)attr.sharedSizeBytes;  // the opt-in limit covers static + dynamic
  if ((size_t)max_dynamic < smem ||
      cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dynamic) != cudaSuccess ||
      cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  if (threads > attr.maxThreadsPerBlock) return 0;
  const int warps = (threads + 31) / 32;
  const int regs_per_warp = bbo::round_up(attr.numRegs, 8) * 32;
  const int by_smem = (int)((size_t)lim.smem_per_sm / (smem + attr.sharedSizeBytes + 1024));  // 1 KB per CTA is reserved
  int by_regs = lim.regs_per_sm / (regs_per_warp * warps);
  // the registers sit in four partitions of a quarter each; warps are dealt to the partitions in turn
  while (by_regs > 1 && (by_regs * warps + 3) / 4 * regs_per_warp > lim.regs_per_sm / 4) --by_regs;
  const int by_tmem = tmem_cols > 0 ? 512 / tmem_cols : 32;
  const int by_threads = 2048 / threads;
  return std::max(0, std::min(std::min(by_smem, by_regs), std::min(std::min(by_tmem, by_threads), 32)));
}

// Plans the launch of fits of padded width Hs.  Threads: one per gradient tile of W1 (8 rows x
// 8 columns) and one per hidden unit.  Sub-tile height: the largest of 32, 16, 8 that fits.
// probe_only: skip the occupancy queries (no CUDA calls), used by the caps query.
int plan_bucket(const DeviceLimits& lim, int n, int d, int C, int K, int Hs, int maxB, bool tracing, bool probe_only,
                Plan* out) {
  const int smem_optin = lim.smem_optin;
  Plan p{};
  p.C = C;
  p.CS = bbo::round_up(C, 4);
  p.dp = bbo::round_up(d, 8);
  p.Hs = Hs;
  const int n_tr_max = K == 1 ? n : n - n / K;  // K == 1: hold-out mode, every row trains
  p.order_bytes = bbo::round_up(2 * n_tr_max, 16);
  p.loss_cap = tracing ? std::min(maxB, n_tr_max) : 0;
  p.n_sort = n_tr_max;
  const int tiles = (p.dp / 8) * (Hs / 8);
  p.NT = bbo::round_up(std::max(std::max(tiles, Hs), 32), 32);
  if (p.NT > bbo::kMaxFitThreads) return BBO_ERR_UNSUPPORTED;
  p.tmem_cols = tiles <= 128 ? 128 : 256;  // 128 columns per group of four tile-owner warps
  const size_t budget = (size_t)smem_optin - 256;  // static block scalars
  for (int TB = 32; TB >= 8; TB >>= 1) {
    const size_t plain = bbo::fit_smem_bytes(d, p.dp, Hs, C, p.CS, TB, p.order_bytes, p.loss_cap, p.n_sort);
    if (plain > budget) continue;
    p.TB = TB;
    p.smem = plain;
    p.per_sm = 1;
    if (probe_only) {
      *out = p;
      return BBO_OK;
    }
    p.kernel = bbo::fit_kernel_for(C, Hs, p.dp);
    if (!p.kernel) return BBO_ERR_UNSUPPORTED;
    p.per_sm = kernel_occupancy(p.kernel, p.NT, plain, p.tmem_cols, lim);
    if (p.per_sm < 1) continue;
    // Pipelined schedule: where the fit sits alone on its SM anyway and batches span several
    // sub-tiles, two extra warps run the output layer of one sub-tile under the gradient tiles of
    // the previous one.  It needs a third row buffer and a second activation buffer.
    if (TB == 32 && p.per_sm == 1 && Hs >= bbo::kPipeHsMin && maxB > TB && bbo::pipe_extra_warps(Hs) == 2) {
      const void* k = bbo::fit_kernel_for(C, Hs, p.dp, true);
      const size_t sm = bbo::fit_smem_bytes(d, p.dp, Hs, C, p.CS, TB, p.order_bytes, p.loss_cap, p.n_sort, true);
      if (k && sm <= budget && kernel_occupancy(k, p.NT + 64, sm, p.tmem_cols, lim) >= 1) {
        p.extra_warps = 2;
        p.NT += 64;
        p.smem = sm;
        p.kernel = k;
      }
    }
    *out = p;
    return BBO_OK;
  }
  return BBO_ERR_UNSUPPORTED;
}

// Where the fits of one evaluation run: the caller's stream plus optional side streams.
struct LaunchEnv {
  DeviceLimits lim;
  cudaStream_t main = nullptr;
  cudaStream_t* aux = nullptr;  // may be null: everything runs on `main`
  int n_aux = 0;
  cudaEvent_t fork = nullptr;
  cudaEvent_t* join = nullptr;
};

struct FitBuffers {  // device scratch of one evaluation
  bbo::Config* configs;
  int2* fits;
  float* fold_scores;
  const int32_t* pi;
  float* trace;
  float* keep_theta;
  const int32_t* config_keys;  // per-configuration keys of the random streams (null: position + base)
};

// Orders the fits for launch.  Grids are dispatched in launch order, so the fits are first cut
// into cost tiers (the costliest tenth, then 20 %, 30 %, 40 % of the fits) and, inside a tier,
// grouped by padded hidden width (widest first) and sorted by descending cost: long fits start
// early whatever their width, and the last launches hold only cheap fits, which keeps the tail
// short.  Cost model (SM cycles, from phase timings): per optimizer step 8000 + 80 H fixed
// (Adam, barriers, chain latencies) plus 2.9 H per row.  One grid per (tier, width) group, on
// the side streams when there are any.
struct HoldoutRows {  // hold-out mode: the rows to score (null Xt = cross-validation)
  const float* Xt = nullptr;
  const float* yt = nullptr;
  int n_test = 0;
};

int launch_all_fits(const LaunchEnv& env, const FitBuffers& buf, const float* Xk, const float* y, int n, int d,
                    int C, int K, int task, const bbo_mlp_config* configs, int n_configs, uint64_t seed,
                    int trace_steps, int maxB, int config_base, int solver, int metric, const HoldoutRows& ho,
                    int* launches, cudaError_t* cuda_err) {
  *cuda_err = cudaSuccess;
  const int n_fits = n_configs * K;
  struct Item { int tier; int Hs; double cost; int id; };
  std::vector<Item> items((size_t)n_fits);
  for (int c = 0; c < n_configs; ++c) {
    const bbo_mlp_config& q = configs[c];
    for (int f = 0; f < K; ++f) {
      int vb, vs;
      bbo::fold_segment(n, K, f, &vb, &vs);
      if (ho.Xt) vs = 0;  // hold-out mode: every row trains
      const double n_tr = n - vs, B = std::min<double>(q.batch_size, n_tr);
      const double steps = (double)q.epochs * std::ceil(n_tr / B);
      const double width = (double)q.hidden * (d + C) / 74.0;  // H for the 64-feature, 10-class shape
      items[(size_t)c * K + f] = {0, bbo::round_up(q.hidden, 8),
                                  steps * (8000.0 + 80.0 * width) + (double)q.epochs * n_tr * 2.9 * width, c * K + f};
    }
  }
  {
    std::vector<int> by_cost((size_t)n_fits);
    for (int i = 0; i < n_fits; ++i) by_cost[i] = i;
    std::stable_sort(by_cost.begin(), by_cost.end(), [&](int a, int b) { return items[a].cost > items[b].cost; });
    for (int r = 0; r < n_fits; ++r) {
      const double q = (double)r / n_fits;
      items[by_cost[r]].tier = q < 0.10 ? 0 : (q < 0.30 ? 1 : (q < 0.60 ? 2 : 3));
    }
  }
  std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
    if (a.tier != b.tier) return a.tier < b.tier;
    return a.Hs != b.Hs ? a.Hs > b.Hs : a.cost > b.cost;
  });
  std::vector<int2> fits((size_t)n_fits);
  for (int i = 0; i < n_fits; ++i) fits[i] = make_int2(items[i].id / K, items[i].id % K);
  // plan every group before anything is enqueued
  struct Group { int begin, count; Plan plan; };
  std::vector<Group> groups;
  for (int i = 0; i < n_fits;) {
    int j = i;
    while (j < n_fits && items[j].Hs == items[i].Hs && items[j].tier == items[i].tier) ++j;
    Group g{i, j - i, {}};
    const int rc = plan_bucket(env.lim, n, d, C, K, items[i].Hs, maxB, trace_steps > 0, false, &g.plan);
    if (rc != BBO_OK) return rc;
    groups.push_back(g);
    i = j;
  }
  cudaError_t e;
  if ((e = cudaMemcpyAsync(buf.configs, configs, sizeof(bbo_mlp_config) * (size_t)n_configs, cudaMemcpyHostToDevice, env.main)) != cudaSuccess ||
      (e = cudaMemcpyAsync(buf.fits, fits.data(), sizeof(int2) * (size_t)n_fits, cudaMemcpyHostToDevice, env.main)) != cudaSuccess) {
    *cuda_err = e;
    return BBO_ERR_CUDA;
  }
  const bool side = env.n_aux > 0 && groups.size() > 1;
  if (side) {
    if ((e = cudaEventRecord(env.fork, env.main)) != cudaSuccess) { *cuda_err = e; return BBO_ERR_CUDA; }
    for (int i = 0; i < env.n_aux; ++i)
      if ((e = cudaStreamWaitEvent(env.aux[i], env.fork, 0)) != cudaSuccess) { *cuda_err = e; return BBO_ERR_CUDA; }
  }
  for (size_t gi = 0; gi < groups.size(); ++gi) {
    const Group& g = groups[gi];
    bbo::FitArgs a{};
    a.X = Xk; a.y = y; a.pi = buf.pi; a.configs = buf.configs; a.fits = buf.fits + g.begin;
    a.fold_scores = buf.fold_scores; a.trace = buf.trace; a.keep_theta = buf.keep_theta;
    a.n_fits = g.count; a.n_configs = n_configs; a.config_base = config_base; a.config_keys = buf.config_keys;
    a.solver = solver; a.metric = metric; a.extra_warps = g.plan.extra_warps;
    a.Xt = ho.Xt; a.yt = ho.yt; a.n_test = ho.n_test;
    a.n = n; a.d = d; a.dp = g.plan.dp; a.C = C; a.CS = g.plan.CS; a.K = K; a.task = task;
    a.Hs = g.plan.Hs; a.TB = g.plan.TB; a.trace_steps = trace_steps; a.loss_cap = g.plan.loss_cap;
    a.order_bytes = g.plan.order_bytes; a.seed = seed;
    a.tmem_cols = g.plan.tmem_cols;
    cudaStream_t s = side ? env.aux[gi % env.n_aux] : env.main;
    void* kargs[] = {&a};
    if ((e = cudaLaunchKernel(g.plan.kernel, dim3(g.count), dim3(g.plan.NT), kargs, g.plan.smem, s)) != cudaSuccess) { *cuda_err = e; return BBO_ERR_CUDA; }
    ++*launches;
  }
  if (side) {
    for (int i = 0; i < env.n_aux; ++i) {
      if ((e = cudaEventRecord(env.join[i], env.aux[i])) != cudaSuccess ||
          (e = cudaStreamWaitEvent(env.main, env.join[i], 0)) != cudaSuccess) { *cuda_err = e; return BBO_ERR_CUDA; }
    }
  }
  return BBO_OK;
}

cudaError_t launch_fold_permutation(int n, uint64_t seed, int32_t* pi, cudaStream_t s) {
  const size_t bytes = 8u * (size_t)bbo::next_pow2(n);
  cudaError_t e = cudaFuncSetAttribute(bbo::fold_permutation_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  bbo::fold_permutation_kernel<<<1, 1024, bytes, s>>>(n, seed, pi);
  return cudaGetLastError();
}

int check_configs(const bbo_mlp_config* cfg, int n_configs, int* maxH, int* maxB) {
  *maxH = 1;
  *maxB = 1;
  for (int c = 0; c < n_configs; ++c) {
    const bbo_mlp_config& q = cfg[c];
    if (q.hidden < 1 || q.batch_size < 1 || q.epochs < 0 || q.epochs >= (1 << 28)) return BBO_ERR_INVALID_ARG;
    if (!(q.alpha >= 0.f) || !std::isfinite(q.alpha) || !(q.lr >= 0.f) || !std::isfinite(q.lr)) return BBO_ERR_INVALID_ARG;
    if (!(q.beta1 >= 0.f && q.beta1 < 1.f) || !(q.beta2 >= 0.f && q.beta2 < 1.f)) return BBO_ERR_INVALID_ARG;
    if (!(q.eps > 0.f) || !std::isfinite(q.eps)) return BBO_ERR_INVALID_ARG;
    *maxH = std::max(*maxH, q.hidden);
    *maxB = std::max(*maxB, q.batch_size);
  }
  return BBO_OK;
}

}  // namespace

extern "C" {

int bbo_mlp_cv_create(const bbo_mlp_cv_options* opt, bbo_mlp_cv** out) {
  if (!out) return BBO_ERR_INVALID_ARG;
  *out = nullptr;
  bbo_mlp_cv_options o{};
  if (opt) o = *opt;
  else o.device = -1;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) {
    cudaGetLastError();
    return BBO_ERR_CUDA;
  }
  int dev = o.device;
  if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) return BBO_ERR_CUDA;
  if (dev >= count || o.n_classes < 0 || o.n_classes > kMaxClasses || o.trace_steps < 0 || o.config_index_base < 0 ||
      o.solver < 0 || o.solver > BBO_SOLVER_SGD || o.metric < 0 || o.metric > BBO_METRIC_ALT ||
      o.variant < 0 || o.variant > BBO_VARIANT_TF32)
    return BBO_ERR_INVALID_ARG;
  if (o.variant == BBO_VARIANT_TF32) return BBO_ERR_UNSUPPORTED;  // not built: it cannot meet the score tolerance (see the header)
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return BBO_ERR_CUDA;
  if (prop.major != 10) return BBO_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
  bbo_mlp_cv* h = new (std::nothrow) bbo_mlp_cv();
  if (!h) return BBO_ERR_OOM;
  h->device = dev;
  h->stream = static_cast<cudaStream_t>(o.stream);
  h->opt = o;
  h->sm_count = prop.multiProcessorCount;
  h->lim.smem_optin = (int)prop.sharedMemPerBlockOptin;
  h->lim.smem_per_sm = (int)prop.sharedMemPerMultiprocessor;
  h->lim.regs_per_sm = prop.regsPerMultiprocessor;
  DeviceGuard g(dev);
  if (cudaEventCreate(&h->ev0) != cudaSuccess || cudaEventCreate(&h->ev1) != cudaSuccess ||
      cudaEventCreate(&h->evf0) != cudaSuccess || cudaEventCreate(&h->evf1) != cudaSuccess) {
    delete h;
    return BBO_ERR_CUDA;
  }
  bool ok = cudaEventCreateWithFlags(&h->fork, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < kAuxStreams && ok; ++i)
    ok = cudaStreamCreateWithFlags(&h->aux[i], cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->join[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    bbo_mlp_cv_destroy(h);
    return BBO_ERR_CUDA;
  }
  *out = h;
  return BBO_OK;
}

int bbo_mlp_cv_destroy(bbo_mlp_cv* h) {
  if (!h) return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  cudaStreamSynchronize(h->stream);
  h->configs.release(); h->fits.release(); h->fold_scores.release(); h->trace.release();
  h->theta.release(); h->xpad.release(); h->xpad_t.release(); h->hx.release(); h->hy.release(); h->hscores.release();
  h->dbg_f.release(); h->pi.release(); h->misc.release(); h->dbg_i.release(); h->dbg_u.release(); h->keys.release();
  if (h->ev0) cudaEventDestroy(h->ev0);
  if (h->ev1) cudaEventDestroy(h->ev1);
  if (h->evf0) cudaEventDestroy(h->evf0);
  if (h->evf1) cudaEventDestroy(h->evf1);
  if (h->fork) cudaEventDestroy(h->fork);
  for (int i = 0; i < kAuxStreams; ++i) {
    if (h->join[i]) cudaEventDestroy(h->join[i]);
    if (h->aux[i]) cudaStreamDestroy(h->aux[i]);
  }
  delete h;
  return BBO_OK;
}

// Shared body of the cross-validation and hold-out evaluations.  Xt == null: K-fold
// cross-validation.  Xt != null: K must be 1; every row of X trains and the n_test rows of
// (Xt, yt) are scored.
static int eval_impl(bbo_mlp_cv* h, const float* X, const float* y, int64_t n64, int32_t d, int32_t task,
                     int32_t K, const bbo_mlp_config* configs, int32_t n_configs, uint64_t seed,
                     float* out_scores, const float* Xt, const float* yt, int64_t n_test64,
                     const int32_t* config_keys = nullptr) {
  if (!h || !X || !y || !configs || !out_scores) return BBO_ERR_INVALID_ARG;
  const bool holdout = Xt != nullptr;
  if (n64 < 2 || d < 1 || n_configs < 1) return BBO_ERR_INVALID_ARG;
  if (holdout ? (K != 1 || !yt || n_test64 < 1) : (K < 2 || K > n64)) return BBO_ERR_INVALID_ARG;
  if (holdout && n_test64 > kMaxRows) return BBO_ERR_UNSUPPORTED;
  if (task != BBO_TASK_CLASSIFICATION && task != BBO_TASK_REGRESSION) return BBO_ERR_INVALID_ARG;
  if (n64 > kMaxRows || (int64_t)n_configs * K > (1 << 30) || (int64_t)n_configs + h->opt.config_index_base >= (1 << 28))
    return BBO_ERR_UNSUPPORTED;
  int maxH, maxB;
  int rc = check_configs(configs, n_configs, &maxH, &maxB);
  if (rc != BBO_OK) return rc;
  if (config_keys)
    for (int c = 0; c < n_configs; ++c)
      if (config_keys[c] < 0 || config_keys[c] >= (1 << 28)) return BBO_ERR_INVALID_ARG;
  // shape against the kernel caps before anything is reserved or enqueued (class count at its largest)
  if (d > kMaxFeatures || maxH > kMaxHidden) return BBO_ERR_UNSUPPORTED;
  {
    Plan probe;
    const int Cmax = task == BBO_TASK_REGRESSION ? 1 : (h->opt.n_classes > 0 ? h->opt.n_classes : 2);
    rc = plan_bucket(h->lim, (int)n64, d, Cmax, K, bbo::round_up(maxH, 8), maxB, h->opt.trace_steps > 0, true, &probe);
    if (rc != BBO_OK) return rc;
  }
  DeviceGuard g(h->device);
  if (!is_device_ptr(X, h->device) || !is_device_ptr(y, h->device) || !is_device_ptr(out_scores, h->device))
    return BBO_ERR_INVALID_ARG;
  if (holdout && (!is_device_ptr(Xt, h->device) || !is_device_ptr(yt, h->device))) return BBO_ERR_INVALID_ARG;
  const int n = (int)n64;
  const int n_test = holdout ? (int)n_test64 : 0;
  cudaStream_t s = h->stream;
  h->cuda_error.clear();
  h->last_fold_count = h->last_trace_count = h->last_theta_count = 0;

  // misc[0] = work counter, misc[1] = max label, misc[2] = bad-label flag
  BBO_CUDA(h, h->misc.reserve(4));
  BBO_CUDA(h, cudaMemsetAsync(h->misc.p, 0, 4 * sizeof(int32_t), s));
  int launches = 0;
  int C = 1;
  if (task == BBO_TASK_CLASSIFICATION) {
    bbo::label_scan_kernel<<<std::min(64, (n + 255) / 256), 256, 0, s>>>(y, n, h->misc.p + 1);
    BBO_CUDA(h, cudaGetLastError());
    ++launches;
    if (holdout) {  // the class count covers the labels of the test rows as well
      bbo::label_scan_kernel<<<std::min(64, (n_test + 255) / 256), 256, 0, s>>>(yt, n_test, h->misc.p + 1);
      BBO_CUDA(h, cudaGetLastError());
      ++launches;
    }
    int32_t info[2];
    BBO_CUDA(h, cudaMemcpyAsync(info, h->misc.p + 1, sizeof(info), cudaMemcpyDeviceToHost, s));
    BBO_CUDA(h, cudaStreamSynchronize(s));
    if (info[1] != 0) return BBO_ERR_INVALID_ARG;
    C = info[0] + 1;
    if (h->opt.n_classes > 0) {
      if (C > h->opt.n_classes) return BBO_ERR_INVALID_ARG;
      C = h->opt.n_classes;
    }
    if (C > kMaxClasses) return BBO_ERR_UNSUPPORTED;
  }

  const bool tracing = h->opt.trace_steps > 0;
  const int dp = bbo::round_up(d, 8);
  const int n_fits = n_configs * K;
  BBO_CUDA(h, h->configs.reserve(n_configs));
  BBO_CUDA(h, h->fits.reserve(n_fits));
  BBO_CUDA(h, h->fold_scores.reserve(n_fits));
  BBO_CUDA(h, h->pi.reserve(n));
  const int32_t* dkeys = nullptr;
  if (config_keys) {
    BBO_CUDA(h, h->keys.reserve(n_configs));
    BBO_CUDA(h, cudaMemcpyAsync(h->keys.p, config_keys, sizeof(int32_t) * (size_t)n_configs, cudaMemcpyHostToDevice, s));
    dkeys = h->keys.p;
  }
  float* trace = nullptr;
  if (tracing) {
    const size_t cnt = (size_t)n_fits * h->opt.trace_steps;
    BBO_CUDA(h, h->trace.reserve(cnt));
    BBO_CUDA(h, cudaMemsetAsync(h->trace.p, 0xFF, cnt * sizeof(float), s));  // NaN padding
    trace = h->trace.p;
  }
  float* keep = nullptr;
  int64_t theta_count = 0;
  if (h->opt.keep_theta) {
    const int H = configs[n_configs - 1].hidden;
    theta_count = (int64_t)d * H + H + (int64_t)H * C + C;
    BBO_CUDA(h, h->theta.reserve((size_t)theta_count));
    keep = h->theta.p;
  }

  BBO_CUDA(h, cudaEventRecord(h->ev0, s));
  const float* Xk = X;
  if (dp != d || (reinterpret_cast<uintptr_t>(X) & 15u) != 0) {
    BBO_CUDA(h, h->xpad.reserve((size_t)n * dp));
    const size_t total = (size_t)n * dp;
    bbo::pad_rows_kernel<<<(int)std::min<size_t>(1024, (total + 255) / 256), 256, 0, s>>>(X, n, d, dp, h->xpad.p);
    BBO_CUDA(h, cudaGetLastError());
    ++launches;
    Xk = h->xpad.p;
  }
  HoldoutRows ho;
  if (holdout) {
    ho.Xt = Xt; ho.yt = yt; ho.n_test = n_test;
    if (dp != d || (reinterpret_cast<uintptr_t>(Xt) & 15u) != 0) {
      const size_t total = (size_t)n_test * dp;
      BBO_CUDA(h, h->xpad_t.reserve(total));
      bbo::pad_rows_kernel<<<(int)std::min<size_t>(1024, (total + 255) / 256), 256, 0, s>>>(Xt, n_test, d, dp, h->xpad_t.p);
      BBO_CUDA(h, cudaGetLastError());
      ++launches;
      ho.Xt = h->xpad_t.p;
    }
  }
  BBO_CUDA(h, launch_fold_permutation(n, seed, h->pi.p, s));
  ++launches;

  LaunchEnv env;
  env.lim = h->lim; env.main = s; env.aux = h->aux; env.n_aux = kAuxStreams;
  env.fork = h->fork; env.join = h->join;
  FitBuffers buf{h->configs.p, h->fits.p, h->fold_scores.p, h->pi.p, trace, keep, dkeys};
  BBO_CUDA(h, cudaEventRecord(h->evf0, s));
  cudaError_t cuda_err = cudaSuccess;
  rc = launch_all_fits(env, buf, Xk, y, n, d, C, K, task, configs, n_configs, seed, h->opt.trace_steps, maxB,
                       h->opt.config_index_base, h->opt.solver, h->opt.metric, ho, &launches, &cuda_err);
  if (rc == BBO_ERR_CUDA) return cuda_fail(h, cuda_err, "launch_all_fits");
  if (rc != BBO_OK) return rc;
  BBO_CUDA(h, cudaEventRecord(h->evf1, s));
  bbo::fold_mean_kernel<<<(n_configs + 127) / 128, 128, 0, s>>>(h->fold_scores.p, n_configs, K, out_scores);
  BBO_CUDA(h, cudaGetLastError());
  ++launches;
  BBO_CUDA(h, cudaEventRecord(h->ev1, s));
  BBO_CUDA(h, cudaStreamSynchronize(s));
  BBO_CUDA(h, cudaEventElapsedTime(&h->last_ms, h->ev0, h->ev1));
  BBO_CUDA(h, cudaEventElapsedTime(&h->last_fit_ms, h->evf0, h->evf1));
  h->last_launches = launches;
  h->last_fold_count = n_fits;
  h->last_trace_count = tracing ? (int64_t)n_fits * h->opt.trace_steps : 0;
  h->last_theta_count = theta_count;
  return BBO_OK;
}

int bbo_mlp_cv_eval(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d, int32_t task, int32_t K,
                    const bbo_mlp_config* configs, int32_t n_configs, uint64_t seed, float* out_scores) {
  return eval_impl(h, X, y, n, d, task, K, configs, n_configs, seed, out_scores, nullptr, nullptr, 0);
}

int bbo_mlp_cv_eval_keyed(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d, int32_t task, int32_t K,
                          const bbo_mlp_config* configs, const int32_t* config_keys, int32_t n_configs, uint64_t seed,
                          float* out_scores) {
  if (!config_keys) return BBO_ERR_INVALID_ARG;
  return eval_impl(h, X, y, n, d, task, K, configs, n_configs, seed, out_scores, nullptr, nullptr, 0, config_keys);
}

int bbo_mlp_cv_eval_holdout(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, const float* Xtest,
                            const float* ytest, int64_t n_test, int32_t d, int32_t task,
                            const bbo_mlp_config* configs, int32_t n_configs, uint64_t seed, float* out_scores) {
  if (!Xtest || !ytest) return BBO_ERR_INVALID_ARG;
  return eval_impl(h, X, y, n, d, task, 1, configs, n_configs, seed, out_scores, Xtest, ytest, n_test);
}

int bbo_mlp_cv_eval_host(bbo_mlp_cv* h, const float* X, const float* y, int64_t n, int32_t d, int32_t task,
                         int32_t K, const bbo_mlp_config* configs, int32_t n_configs, uint64_t seed,
                         float* out_scores) {
  if (!h || !X || !y || !configs || !out_scores || n < 2 || d < 1 || n_configs < 1) return BBO_ERR_INVALID_ARG;
  if (n > kMaxRows) return BBO_ERR_UNSUPPORTED;
  DeviceGuard g(h->device);
  BBO_CUDA(h, h->hx.reserve((size_t)n * d));
  BBO_CUDA(h, h->hy.reserve((size_t)n));
  BBO_CUDA(h, h->hscores.reserve((size_t)n_configs));
  BBO_CUDA(h, cudaMemcpyAsync(h->hx.p, X, sizeof(float) * (size_t)n * d, cudaMemcpyHostToDevice, h->stream));
  BBO_CUDA(h, cudaMemcpyAsync(h->hy.p, y, sizeof(float) * (size_t)n, cudaMemcpyHostToDevice, h->stream));
  const int rc = bbo_mlp_cv_eval(h, h->hx.p, h->hy.p, n, d, task, K, configs, n_configs, seed, h->hscores.p);
  if (rc != BBO_OK) return rc;
  BBO_CUDA(h, cudaMemcpyAsync(out_scores, h->hscores.p, sizeof(float) * (size_t)n_configs, cudaMemcpyDeviceToHost, h->stream));
  BBO_CUDA(h, cudaStreamSynchronize(h->stream));
  return BBO_OK;
}

static int copy_back(bbo_mlp_cv* h, const float* src, int64_t have, float* host_out, int64_t count) {
  if (!h || !host_out) return BBO_ERR_INVALID_ARG;
  if (have == 0 || count != have) return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  BBO_CUDA(h, cudaMemcpyAsync(host_out, src, sizeof(float) * (size_t)count, cudaMemcpyDeviceToHost, h->stream));
  BBO_CUDA(h, cudaStreamSynchronize(h->stream));
  return BBO_OK;
}

int bbo_mlp_cv_fold_scores(bbo_mlp_cv* h, float* host_out, int64_t count) {
  return h ? copy_back(h, h->fold_scores.p, h->last_fold_count, host_out, count) : BBO_ERR_INVALID_ARG;
}
int bbo_mlp_cv_loss_trace(bbo_mlp_cv* h, float* host_out, int64_t count) {
  return h ? copy_back(h, h->trace.p, h->last_trace_count, host_out, count) : BBO_ERR_INVALID_ARG;
}
int bbo_mlp_cv_debug_theta(bbo_mlp_cv* h, float* host_out, int64_t count) {
  return h ? copy_back(h, h->theta.p, h->last_theta_count, host_out, count) : BBO_ERR_INVALID_ARG;
}

int bbo_mlp_cv_debug_indices(bbo_mlp_cv* h, int64_t n64, int32_t K, uint64_t seed, int32_t config, int32_t fold,
                             int32_t epoch, int32_t* host_fold_of_row, int32_t* host_order) {
  if (!h || n64 < 2 || K < 2 || K > n64 || fold < 0 || fold >= K || config < 0 || epoch < 0) return BBO_ERR_INVALID_ARG;
  if (n64 > kMaxRows || n64 > 65535) return BBO_ERR_UNSUPPORTED;
  const int n = (int)n64;
  DeviceGuard g(h->device);
  cudaStream_t s = h->stream;
  BBO_CUDA(h, h->pi.reserve(n));
  BBO_CUDA(h, h->dbg_i.reserve(2 * (size_t)n));
  BBO_CUDA(h, launch_fold_permutation(n, seed, h->pi.p, s));
  int vb, vs;
  bbo::fold_segment(n, K, fold, &vb, &vs);
  const int n_tr = n - vs;
  const size_t bytes = (size_t)bbo::round_up(2 * n_tr, 16) + bbo::sort_scratch_bytes(n_tr);
  BBO_CUDA(h, cudaFuncSetAttribute(bbo::debug_order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  bbo::debug_order_kernel<<<1, 256, bytes, s>>>(n, K, seed, h->pi.p, config, fold, epoch, h->dbg_i.p, h->dbg_i.p + n);
  BBO_CUDA(h, cudaGetLastError());
  if (host_fold_of_row)
    BBO_CUDA(h, cudaMemcpyAsync(host_fold_of_row, h->dbg_i.p, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost, s));
  if (host_order)
    BBO_CUDA(h, cudaMemcpyAsync(host_order, h->dbg_i.p + n, sizeof(int32_t) * (size_t)n_tr, cudaMemcpyDeviceToHost, s));
  BBO_CUDA(h, cudaStreamSynchronize(s));
  return BBO_OK;
}

int bbo_mlp_cv_debug_rng(bbo_mlp_cv* h, uint64_t seed, const uint32_t* counters, int64_t count, uint32_t* out) {
  if (!h || !counters || !out || count < 1) return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  cudaStream_t s = h->stream;
  BBO_CUDA(h, h->dbg_u.reserve(9 * (size_t)count));
  BBO_CUDA(h, cudaMemcpyAsync(h->dbg_u.p, counters, sizeof(uint32_t) * 5 * (size_t)count, cudaMemcpyHostToDevice, s));
  bbo::debug_rng_kernel<<<(int)std::min<int64_t>(1024, (count + 255) / 256), 256, 0, s>>>(seed, h->dbg_u.p, count, h->dbg_u.p + 5 * count);
  BBO_CUDA(h, cudaGetLastError());
  BBO_CUDA(h, cudaMemcpyAsync(out, h->dbg_u.p + 5 * count, sizeof(uint32_t) * 4 * (size_t)count, cudaMemcpyDeviceToHost, s));
  BBO_CUDA(h, cudaStreamSynchronize(s));
  return BBO_OK;
}

int bbo_mlp_cv_debug_exp(bbo_mlp_cv* h, const float* x, int64_t count, float* out) {
  if (!h || !x || !out || count < 1) return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  cudaStream_t s = h->stream;
  BBO_CUDA(h, h->dbg_f.reserve(2 * (size_t)count));
  BBO_CUDA(h, cudaMemcpyAsync(h->dbg_f.p, x, sizeof(float) * (size_t)count, cudaMemcpyHostToDevice, s));
  bbo::debug_exp_kernel<<<(int)std::min<int64_t>(1024, (count + 255) / 256), 256, 0, s>>>(h->dbg_f.p, count, h->dbg_f.p + count);
  BBO_CUDA(h, cudaGetLastError());
  BBO_CUDA(h, cudaMemcpyAsync(out, h->dbg_f.p + count, sizeof(float) * (size_t)count, cudaMemcpyDeviceToHost, s));
  BBO_CUDA(h, cudaStreamSynchronize(s));
  return BBO_OK;
}

int bbo_mlp_cv_debug_fast_math(bbo_mlp_cv* h, int32_t mode, uint64_t seed, uint64_t first, uint64_t count,
                               uint64_t* host_out4) {
  if (!h || !host_out4 || count < 1 || (mode < 0 || mode > 3)) return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  cudaStream_t s = h->stream;
  BBO_CUDA(h, h->dbg_u.reserve(8));
  BBO_CUDA(h, cudaMemsetAsync(h->dbg_u.p, 0, 32, s));
  bbo::debug_fast_math_kernel<<<h->sm_count * 8, 256, 0, s>>>(mode, seed, first, count, reinterpret_cast<unsigned long long*>(h->dbg_u.p));
  BBO_CUDA(h, cudaGetLastError());
  BBO_CUDA(h, cudaMemcpyAsync(host_out4, h->dbg_u.p, 32, cudaMemcpyDeviceToHost, s));
  BBO_CUDA(h, cudaStreamSynchronize(s));
  return BBO_OK;
}

int bbo_mlp_cv_debug_ffma_peak(bbo_mlp_cv* h, int32_t threads_per_sm, int32_t iters, float* tflops) {
  if (!h || !tflops || threads_per_sm < 32 || threads_per_sm > 1024 || threads_per_sm % 32 != 0 || iters < 1)
    return BBO_ERR_INVALID_ARG;
  DeviceGuard g(h->device);
  cudaStream_t s = h->stream;
  BBO_CUDA(h, h->dbg_f.reserve((size_t)h->sm_count * threads_per_sm));
  bbo::ffma_peak_kernel<<<h->sm_count, threads_per_sm, 0, s>>>(h->dbg_f.p, 100);  // warm-up
  BBO_CUDA(h, cudaEventRecord(h->ev0, s));
  bbo::ffma_peak_kernel<<<h->sm_count, threads_per_sm, 0, s>>>(h->dbg_f.p, iters);
  BBO_CUDA(h, cudaEventRecord(h->ev1, s));
  BBO_CUDA(h, cudaGetLastError());
  BBO_CUDA(h, cudaStreamSynchronize(s));
  float ms = 0.f;
  BBO_CUDA(h, cudaEventElapsedTime(&ms, h->ev0, h->ev1));
  *tflops = (float)(2.0 * 16.0 * (double)iters * threads_per_sm * h->sm_count / (ms * 1e-3) / 1e12);
  return BBO_OK;
}

int bbo_mlp_cv_query_caps(bbo_mlp_cv* h, int32_t d, int32_t n_classes, int32_t* max_n, int32_t* max_d,
                          int32_t* max_hidden, int32_t* max_classes) {
  if (!h || d < 1 || n_classes < 1 || n_classes > kMaxClasses) return BBO_ERR_INVALID_ARG;
  if (max_n) *max_n = kMaxRows;
  if (max_classes) *max_classes = kMaxClasses;
  // widest hidden layer for (d, C) on a 1797-row, 5-fold problem with the smallest sub-tile
  auto fits_H = [&](int dd, int H) {
    Plan p;
    return plan_bucket(h->lim, 1797, dd, n_classes, 5, bbo::round_up(H, 8), 1, false, true, &p) == BBO_OK;
  };
  if (max_hidden) {
    int lo = 0, hi = 4096;
    while (lo < hi) {
      const int mid = (lo + hi + 1) / 2;
      if (fits_H(d, mid)) lo = mid; else hi = mid - 1;
    }
    *max_hidden = lo;
  }
  if (max_d) {
    int lo = 0, hi = 16384;
    while (lo < hi) {
      const int mid = (lo + hi + 1) / 2;
      if (fits_H(mid, 1)) lo = mid; else hi = mid - 1;
    }
    *max_d = lo;
  }
  return BBO_OK;
}

int bbo_mlp_cv_last_timing(bbo_mlp_cv* h, float* total_ms, float* fit_ms, int32_t* n_launches) {
  if (!h) return BBO_ERR_INVALID_ARG;
  if (total_ms) *total_ms = h->last_ms;
  if (fit_ms) *fit_ms = h->last_fit_ms;
  if (n_launches) *n_launches = h->last_launches;
  return BBO_OK;
}

const char* bbo_mlp_cv_strerror(int code) {
  switch (code) {
    case BBO_OK: return "ok";
    case BBO_ERR_INVALID_ARG: return "invalid argument";
    case BBO_ERR_UNSUPPORTED: return "shape or device not supported";
    case BBO_ERR_CUDA: return "CUDA runtime error";
    case BBO_ERR_TIMEOUT: return "device-side wait timed out";
    case BBO_ERR_OOM: return "out of device memory";
    case BBO_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the allocation-free entry point";
    default: return "unknown status";
  }
}

const char* bbo_mlp_cv_last_cuda_error(bbo_mlp_cv* h) { return h ? h->cuda_error.c_str() : ""; }

}  // extern "C"

// ---------------------------------------------------------------------------------------
// Allocation-free evaluation: every working buffer is carved out of one array that is part
// of the library image.  In host code the name `g_static_scratch` is only a handle for the
// runtime, not a device address; the address comes from cudaGetSymbolAddress, once per
// device, and that pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[BBO_STATIC_SCRATCH_BYTES];

namespace {

struct StaticDevice {
  bool ready = false;
  unsigned char* base = nullptr;
  int sm_count = 0, major = 0;
  DeviceLimits lim;
};
constexpr int kMaxDevices = 64;
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mutex;
thread_local std::string g_static_error;  // text of the last CUDA error of bbo_mlp_cv_eval_static on this thread

int static_fail(cudaError_t e, const char* what) {
  g_static_error = std::string(what) + ": " + cudaGetErrorString(e);
  return e == cudaErrorMemoryAllocation ? BBO_ERR_OOM : BBO_ERR_CUDA;
}

// One-off set-up for the current device: device address of the scratch array and the
// device limits the launch plan needs.
int static_device_setup(int dev, StaticDevice* out) {
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticDevice& sd = g_static_dev[dev];
  if (!sd.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return BBO_ERR_CUDA;
    }
    if (cudaDeviceGetAttribute(&sd.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.lim.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.lim.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.lim.regs_per_sm, cudaDevAttrMaxRegistersPerMultiprocessor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
      cudaGetLastError();
      return BBO_ERR_CUDA;
    }
    sd.base = static_cast<unsigned char*>(ptr);
    sd.ready = true;
  }
  *out = sd;
  return BBO_OK;
}

}  // namespace

extern "C" int bbo_mlp_cv_eval_static(void* stream, const float* X, const float* y, int64_t n64, int32_t d,
                                      int32_t task, int32_t K, int32_t n_classes, const bbo_mlp_config* configs,
                                      int32_t n_configs, uint64_t seed, float* out_scores) {
  g_static_error.clear();
  if (!X || !y || !configs || !out_scores) return BBO_ERR_INVALID_ARG;
  if (n64 < 2 || d < 1 || K < 2 || K > n64 || n_configs < 1 || n_classes < 0 || n_classes > kMaxClasses)
    return BBO_ERR_INVALID_ARG;
  if (task != BBO_TASK_CLASSIFICATION && task != BBO_TASK_REGRESSION) return BBO_ERR_INVALID_ARG;
  const int64_t dp64 = (int64_t)(d + 7) / 8 * 8;
  if (n64 > BBO_STATIC_MAX_ROWS || n64 * dp64 > BBO_STATIC_MAX_X_FLOATS || n_configs > BBO_STATIC_MAX_CONFIGS ||
      (int64_t)n_configs * K > BBO_STATIC_MAX_FITS)
    return BBO_ERR_TOO_LARGE;
  int maxH, maxB;
  int rc = check_configs(configs, n_configs, &maxH, &maxB);
  if (rc != BBO_OK) return rc;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BBO_ERR_CUDA;
  StaticDevice sd;
  rc = static_device_setup(dev, &sd);
  if (rc != BBO_OK) return rc;
  if (sd.major != 10) return BBO_ERR_UNSUPPORTED;
  if (!is_device_ptr(X, dev) || !is_device_ptr(y, dev) || !is_device_ptr(out_scores, dev)) return BBO_ERR_INVALID_ARG;
  const int n = (int)n64;
  const int n_fits = n_configs * K;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // carve the array: [misc 256 B][pi][configs][fits][fold scores][padded X]
  unsigned char* p = sd.base;
  int32_t* misc = reinterpret_cast<int32_t*>(p);            p += 256;
  int32_t* pi = reinterpret_cast<int32_t*>(p);              p += 4 * (size_t)BBO_STATIC_MAX_ROWS;
  bbo::Config* dcfg = reinterpret_cast<bbo::Config*>(p);    p += 32 * (size_t)BBO_STATIC_MAX_CONFIGS;
  int2* dfits = reinterpret_cast<int2*>(p);                 p += 8 * (size_t)BBO_STATIC_MAX_FITS;
  float* fold_scores = reinterpret_cast<float*>(p);         p += 4 * (size_t)BBO_STATIC_MAX_FITS;
  float* xpad = reinterpret_cast<float*>(p);

  // the work counter and the label summary must start from zero; everything else is
  // fully rewritten before it is read
  if (cudaMemsetAsync(misc, 0, 256, s) != cudaSuccess) return BBO_ERR_CUDA;
  int C = 1;
  if (task == BBO_TASK_CLASSIFICATION) {
    bbo::label_scan_kernel<<<std::min(64, (n + 255) / 256), 256, 0, s>>>(y, n, misc + 1);
    int32_t info[2];
    if (cudaGetLastError() != cudaSuccess ||
        cudaMemcpyAsync(info, misc + 1, sizeof(info), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
      return BBO_ERR_CUDA;
    if (info[1] != 0) return BBO_ERR_INVALID_ARG;
    C = info[0] + 1;
    if (n_classes > 0) {
      if (C > n_classes) return BBO_ERR_INVALID_ARG;
      C = n_classes;
    }
    if (C > kMaxClasses) return BBO_ERR_UNSUPPORTED;
  }

  const int dp = bbo::round_up(d, 8);
  const float* Xk = X;
  if (dp != d || (reinterpret_cast<uintptr_t>(X) & 15u) != 0) {
    const size_t total = (size_t)n * dp;
    bbo::pad_rows_kernel<<<(int)std::min<size_t>(1024, (total + 255) / 256), 256, 0, s>>>(X, n, d, dp, xpad);
    if (cudaGetLastError() != cudaSuccess) return BBO_ERR_CUDA;
    Xk = xpad;
  }
  if (launch_fold_permutation(n, seed, pi, s) != cudaSuccess) return BBO_ERR_CUDA;
  LaunchEnv env;  // no side streams: creating them would be a resource allocation
  env.lim = sd.lim;
  env.main = s;
  FitBuffers buf{dcfg, dfits, fold_scores, pi, nullptr, nullptr, nullptr};
  int launches = 0;
  cudaError_t cuda_err = cudaSuccess;
  rc = launch_all_fits(env, buf, Xk, y, n, d, C, K, task, configs, n_configs, seed, 0, maxB, 0, BBO_SOLVER_ADAM,
                       BBO_METRIC_DEFAULT, HoldoutRows{}, &launches, &cuda_err);
  if (rc == BBO_ERR_CUDA) return static_fail(cuda_err, "launch_all_fits");
  if (rc != BBO_OK) return rc;
  bbo::fold_mean_kernel<<<(n_configs + 127) / 128, 128, 0, s>>>(fold_scores, n_configs, K, out_scores);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return static_fail(e, "fold mean / stream synchronisation");
  return BBO_OK;
}

extern "C" const char* bbo_mlp_cv_static_last_cuda_error(void) { return g_static_error.c_str(); }
