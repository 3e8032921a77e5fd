// Warp-specialised schedule of one (configuration, fold) fit (paper sec. 2: the evaluated function
// is a cross-validation score; Table 1: MLP-adam / MLP-sgd; sec. 5: evaluation runs on the GPU).
//
// Same arithmetic contract as fit_kernel.cuh: every accumulator has one owner thread and
// receives its terms in one fixed order, so the results are bit-identical to the phased kernel.
// What changes is who works when.  The warps of the CTA are split into four roles that run
// concurrently on different sub-tiles (TB rows) of the minibatch, handing buffers to one another
// through shared-memory barriers:
//   H  hidden layer: 8x8 register tiles of A1 = relu(X W1 + b1); its first warp also issues the
//      bulk row copies (global -> shared, completing on a barrier) of the next sub-tile
//   O  output layer, softmax / residual, loss derivative (one lane per row, all classes)
//   U  one thread per pair of hidden units: gW2, delta1 in place over A1, gb1 (and gb2)
//   G  8x8 register tiles of the W1 gradient, kept in registers across the sub-tiles of a step;
//      the owner applies L2 + Adam to exactly its elements, with the first and second moments of
//      W1 held in tensor memory (each thread stores and reloads its own 128 words once per step)
// In steady state H works on sub-tile t+1, O and U on t, G on t-1.  Parameters W1, b1, W2, b2
// stay in shared memory; the moments of b1, W2, b2 too.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "device_math.cuh"
#include "fit_common.cuh"
#include "fit_kernel.cuh"
#include "sm100_primitives.cuh"

namespace bbo {

constexpr int kWaitLimit = 1 << 20;  // polls (each a suspension of up to a microsecond) of one barrier wait before the fit gives up

struct RoleShared {
  uint64_t xfull[kNX], xfree[kNX], a1ready[kNA], a1free[kNA], d1ready[kNA], d2ready[kND], d2free[kND], params;
  float step[2];  // Adam step size by step parity (written one step ahead of its readers)
  int correct;
  float sq;
  float red[32];
  uint32_t tmem_base;
  volatile int abort;  // set when a wait ran out; every later wait returns at once
#ifdef BBO_PHASE_TIMERS
  long long t_wait[4][4];  // [role][wait kind]
  long long t_sort, t_train, t_adam[2];
#endif
};

#ifdef BBO_PHASE_TIMERS
#define BBO_ROLE_WAIT(kind, call) do { const long long tw_ = clock64(); call; if (rw == 0 && lane == 0) sh.t_wait[role][kind] += clock64() - tw_; } while (0)
#else
#define BBO_ROLE_WAIT(kind, call) do { call; } while (0)
#endif

// Waits for the phase of `parity` of `bar`.  Gives up after kWaitLimit polls (or as soon as
// another thread has given up), setting the abort flag; the caller then skips its work but keeps
// walking the schedule so that every block-wide barrier is still reached by all threads.
__device__ __forceinline__ bool role_wait(RoleShared& sh, uint64_t* bar, uint32_t parity) {
  for (int i = 0; i < kWaitLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(100);
    if ((i & 255) == 255 && sh.abort) return false;
  }
  sh.abort = 1;
  return false;
}

// A1 = relu(xs W1 + b1) for nb rows: each thread owns tiles of 8 rows x 8 columns (columns
// jA..jA+3 and jB..jB+3, jB = jA + Hs/2), k ascending from the bias.  hid / hthreads: index of
// the calling thread among the threads that share the work.
__device__ __forceinline__ void hidden_tiles(const float* W, const Layout& L, const float* xs, float* A1b, int d, int dp, int Hs,
                                             int nb, int hid, int hthreads) {
  const int CG = Hs >> 3, n_tiles = ((nb + 7) >> 3) * CG, half = Hs >> 1, d2 = d >> 1;
  for (int t = hid; t < n_tiles; t += hthreads) {
    const int rg = t / CG, cg = t - rg * CG;
    const int r0 = rg << 3, jA = cg << 2, jB = half + jA;
    float acc[8][8];
    {
      const float4 ba = *reinterpret_cast<const float4*>(W + L.ob1 + jA), bb = *reinterpret_cast<const float4*>(W + L.ob1 + jB);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc[i][0] = ba.x; acc[i][1] = ba.y; acc[i][2] = ba.z; acc[i][3] = ba.w;
        acc[i][4] = bb.x; acc[i][5] = bb.y; acc[i][6] = bb.z; acc[i][7] = bb.w;
      }
    }
    const float* xr = xs + r0 * dp;
    const float* wa = W + L.oW1 + jA;
    const float* wb = W + L.oW1 + jB;
#pragma unroll 1
    for (int k2 = 0; k2 < d2; ++k2) {
      float2 xv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) xv[i] = *reinterpret_cast<const float2*>(xr + i * dp + 2 * k2);
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        const float4 va = *reinterpret_cast<const float4*>(wa + (2 * k2 + kk) * Hs);
        const float4 vb = *reinterpret_cast<const float4*>(wb + (2 * k2 + kk) * Hs);
        const float wv[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float x = kk == 0 ? xv[i].x : xv[i].y;
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[i][j] = __fmaf_rn(x, wv[j], acc[i][j]);
        }
      }
    }
    for (int k = d2 << 1; k < d; ++k) {
      const float4 va = *reinterpret_cast<const float4*>(wa + k * Hs);
      const float4 vb = *reinterpret_cast<const float4*>(wb + k * Hs);
      const float wv[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float x = xr[i * dp + k];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = __fmaf_rn(x, wv[j], acc[i][j]);
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float4 o, p;
      o.x = acc[i][0] > 0.f ? acc[i][0] : 0.f; o.y = acc[i][1] > 0.f ? acc[i][1] : 0.f;
      o.z = acc[i][2] > 0.f ? acc[i][2] : 0.f; o.w = acc[i][3] > 0.f ? acc[i][3] : 0.f;
      p.x = acc[i][4] > 0.f ? acc[i][4] : 0.f; p.y = acc[i][5] > 0.f ? acc[i][5] : 0.f;
      p.z = acc[i][6] > 0.f ? acc[i][6] : 0.f; p.w = acc[i][7] > 0.f ? acc[i][7] : 0.f;
      *reinterpret_cast<float4*>(A1b + (r0 + i) * L.WP + jA) = o;
      *reinterpret_cast<float4*>(A1b + (r0 + i) * L.WP + jB) = p;
    }
  }
}

// Output layer of one row held by one thread: z[o] = b2[o] + sum_j a1[j] W2[j][o], j ascending.
// W2 is class-major with pitch L.WP, so one 16-byte load per class (the same address in every
// lane) feeds four steps of its chain; the operands of the next four steps are fetched before the
// current multiply-adds are issued.  arow: the row's activations (padded by four floats).
template <int CT>
__device__ __forceinline__ void row_logits(const float* W, const Layout& L, int H, const float* arow, float (&z)[CT]) {
  const float* w2 = W + L.oW2;
#pragma unroll
  for (int o = 0; o < CT; ++o) z[o] = W[L.ob2 + o];
  int j = 0;
  float4 a_nx = *reinterpret_cast<const float4*>(arow);
  float4 w_nx[CT];
#pragma unroll
  for (int o = 0; o < CT; ++o) w_nx[o] = *reinterpret_cast<const float4*>(w2 + o * L.WP);
#pragma unroll 1
  for (; j + 4 <= H; j += 4) {
    const float4 av = a_nx;
    float4 w[CT];
#pragma unroll
    for (int o = 0; o < CT; ++o) w[o] = w_nx[o];
    a_nx = *reinterpret_cast<const float4*>(arow + j + 4);  // rows are padded: stays inside the row
#pragma unroll
    for (int o = 0; o < CT; ++o) w_nx[o] = *reinterpret_cast<const float4*>(w2 + o * L.WP + j + 4);
#pragma unroll
    for (int o = 0; o < CT; ++o) z[o] = __fmaf_rn(av.x, w[o].x, z[o]);
#pragma unroll
    for (int o = 0; o < CT; ++o) z[o] = __fmaf_rn(av.y, w[o].y, z[o]);
#pragma unroll
    for (int o = 0; o < CT; ++o) z[o] = __fmaf_rn(av.z, w[o].z, z[o]);
#pragma unroll
    for (int o = 0; o < CT; ++o) z[o] = __fmaf_rn(av.w, w[o].w, z[o]);
  }
  for (; j < H; ++j) {
    const float av = arow[j];
#pragma unroll
    for (int o = 0; o < CT; ++o) z[o] = __fmaf_rn(av, w2[o * L.WP + j], z[o]);
  }
}

// Softmax statistics of one row: running maximum (strict >) and denominator, both over the
// classes in ascending order.
template <int CT>
__device__ __forceinline__ void row_softmax(const float (&z)[CT], float& mx, float (&ex)[CT], float& sum) {
  mx = z[0];
#pragma unroll
  for (int o = 1; o < CT; ++o) if (z[o] > mx) mx = z[o];
#pragma unroll
  for (int o = 0; o < CT; ++o) ex[o] = spec_expf(__fsub_rn(z[o], mx));
  sum = 0.f;
#pragma unroll
  for (int o = 0; o < CT; ++o) sum = __fadd_rn(sum, ex[o]);
}

// Loss derivative of one row, written to d2row[0..CT); loss_out (may be null) receives the row's loss.
template <int CT>
__device__ __forceinline__ void row_loss_derivative(int task, const float (&z)[CT], float yv, float invB, float* d2row, float* loss_out) {
  if (task == 0) {
    const int label = (int)yv;
    float mx, sum, ex[CT];
    row_softmax<CT>(z, mx, ex, sum);
    // probabilities: branch-free division first; the IEEE routine only where it cannot be certified
    float pr[CT];
    uint32_t safe = 1u;
#pragma unroll
    for (int o = 0; o < CT; ++o) pr[o] = softmax_ratio_fast(ex[o], sum, safe);
    if (!safe) {
#pragma unroll
      for (int o = 0; o < CT; ++o) pr[o] = sum != sum ? sum : __fdiv_rn(ex[o], sum);  // NaN row: skip the library's special cases
    }
    float zl = 0.f;
#pragma unroll
    for (int o = 0; o < CT; ++o) {
      d2row[o] = __fmul_rn(__fsub_rn(pr[o], o == label ? 1.0f : 0.0f), invB);
      if (o == label) zl = z[o];
    }
    if (loss_out) *loss_out = __fsub_rn(logf(sum), __fsub_rn(zl, mx));
    return;
  }
  const float r = __fsub_rn(z[0], yv);
  if (loss_out) *loss_out = __fmul_rn(__fmul_rn(0.5f, r), r);
  d2row[0] = __fmul_rn(r, invB);
}

// Position of a sub-tile inside an epoch: minibatch start s0 and row offset t0 inside it.
struct TileCursor {
  int s0, t0;
  __device__ __forceinline__ bool valid(int n_tr) const { return s0 < n_tr; }
  __device__ __forceinline__ int rows(int n_tr, int B, int TB) const {
    const int Bs = (n_tr - s0) < B ? (n_tr - s0) : B;
    return (Bs - t0) < TB ? (Bs - t0) : TB;
  }
  __device__ __forceinline__ void advance(int n_tr, int B, int TB) {
    const int Bs = (n_tr - s0) < B ? (n_tr - s0) : B;
    t0 += TB;
    if (t0 >= Bs) { s0 += B; t0 = 0; }
  }
};

// The whole fit.  CT: class count.  HSC / DPC: compile-time padded hidden width / feature count
// (0 = run-time).
// RB: the CTA has 512 threads, the roles sit on warp-group boundaries (G: warps 0-7, H: 8-11,
// O: 12-13, U: 14-15) and the 65,536 registers are re-divided between them (setmaxnreg) for the
// training loop: 136 per G thread (gradient tile, moments in flight), 120 per H, O and U thread.
template <int CT, int HSC, int DPC, bool RB>
__device__ __forceinline__ void run_fit_roles(const FitArgs& a, int q, float* smem, RoleShared& sh) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int2 cf = a.fits[q];
  const int config = cf.x, fold = cf.y;
  const uint32_t rng_config = (uint32_t)(config + a.config_base);
  const Config c = a.configs[config];
  const int H = c.hidden, d = a.d, CS = a.CS, TB = a.TB;
  const int dp = DPC ? DPC : a.dp;
  const int Hs = HSC ? HSC : a.Hs;
  const Layout L(d, Hs, CT, CS);
  const bool holdout = a.Xt != nullptr;
  const uint32_t rng_fold = holdout ? kHoldoutFoldKey : (uint32_t)fold;
  int vb = 0, vs = 0;
  if (!holdout) fold_segment(a.n, a.K, fold, &vb, &vs);
  const int n_tr = a.n - vs;
  if (holdout) vs = a.n_test;
  const int B = c.batch_size < n_tr ? c.batch_size : n_tr;

  // ---- roles ----
  const int wH0 = a.nG, wO0 = wH0 + a.nH, wU0 = wO0 + a.nO;
  const int role = warp < wH0 ? 0 : (warp < wO0 ? 1 : (warp < wU0 ? 2 : 3));  // G, H, O, U
  const int rw = warp - (role == 0 ? 0 : (role == 1 ? wH0 : (role == 2 ? wO0 : wU0)));  // warp index inside the role
  const int rid = rw * 32 + lane;                                                       // thread index inside the role

  // ---- shared memory ----
  float* W = smem;
  float* Msm = W + L.PS - L.ob1;          // moments of b1, W2, b2: Msm[off], Vsm[off] for off >= ob1
  float* Vsm = Msm + L.PT;
  char* p = reinterpret_cast<char*>(W + L.PS + 2 * L.PT);
  uint16_t* order = reinterpret_cast<uint16_t*>(p); p += a.order_bytes;
  float* lossb = reinterpret_cast<float*>(p);       p += round_up(4 * a.loss_cap, 16);
  float* D2 = reinterpret_cast<float*>(p);          p += 4 * kND * TB * CS;
  p = reinterpret_cast<char*>(smem) + ((p - reinterpret_cast<char*>(smem)) + 127) / 128 * 128;
  float* Xs = reinterpret_cast<float*>(p);
  float* A1 = Xs + kNX * TB * dp;
  void* keys = p;
  const uint32_t row_bytes = 4u * (uint32_t)dp;

  // ---- initialisation: Glorot-uniform parameters, zero moments, barriers, tensor memory ----
  for (int i = tid; i < L.PS + 2 * L.PT; i += nt) W[i] = 0.f;
  if (tid == 0) {
    for (int i = 0; i < kNX; ++i) { mbar_init(&sh.xfull[i], 1); mbar_init(&sh.xfree[i], a.nG); }
    for (int i = 0; i < kNA; ++i) { mbar_init(&sh.a1ready[i], a.nH); mbar_init(&sh.a1free[i], a.nG); mbar_init(&sh.d1ready[i], a.nU); }
    for (int i = 0; i < kND; ++i) { mbar_init(&sh.d2ready[i], a.nO); mbar_init(&sh.d2free[i], a.nU); }
    mbar_init(&sh.params, a.nG + a.nU);
    mbar_init_fence();
    sh.abort = 0;
  }
  if (warp == 0) tmem_alloc(&sh.tmem_base, (uint32_t)a.tmem_cols);
  tmem_fence_before_sync();
  __syncthreads();
  tmem_fence_after_sync();
  {
    const float bound1 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(d + H)));
    const float bound2 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(H + CT)));
    const int n1 = d * H, n2 = H * CT;
    for (int blk = tid; blk < ((n1 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 0u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n1) { const int k = idx / H, j = idx - k * H; W[L.oW1 + k * Hs + j] = glorot_value(word_of(r, w), bound1); }
      }
    }
    for (int blk = tid; blk < ((H + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 1u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int j = 4 * blk + w; if (j < H) W[L.ob1 + j] = glorot_value(word_of(r, w), bound1); }
    }
    for (int blk = tid; blk < ((n2 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 2u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n2) { const int j = idx / CT, o = idx - j * CT; W[L.oW2 + o * L.WP + j] = glorot_value(word_of(r, w), bound2); }
      }
    }
    for (int blk = tid; blk < ((CT + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 3u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int o = 4 * blk + w; if (o < CT) W[L.ob2 + o] = glorot_value(word_of(r, w), bound2); }
    }
  }
  // tensor-memory home of this thread's W1 moments: lanes of the warp's quarter, 128 columns per
  // group of four G warps; first moments in columns 0..63 (row i of the tile at 8 i), second
  // moments in 64..127
  const uint32_t tm = sh.tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + 128u * (uint32_t)(warp >> 2);
  if (role == 0) {
    const float zero8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 16; ++i) tmem_store8(tm + 8u * i, zero8);
    tmem_wait_stores();
  }
  __syncthreads();

  // ---- per-role constants ----
  const int KG = dp >> 3, JG8 = Hs >> 3;
  const bool has_tile = role == 0 && rid < KG * JG8;
  const int kg = has_tile ? rid / JG8 : 0, jg = has_tile ? rid - kg * JG8 : 0;
  const int k0 = kg << 3, jA = jg << 2, jB = (jg + JG8) << 2;
  const int hthreads = a.nH * 32;
  constexpr int UPT = units_per_thread(CT);            // U: hidden units uj .. uj + UPT - 1 per thread
  const int uj = UPT * rid;
  const bool unit_any = role == 3 && uj < H;
  const int ob_first = Hs / UPT;                       // U: threads ob_first .. ob_first + CT - 1 own gb2 / b2
  const bool o_role = role == 3 && rid >= ob_first && rid < ob_first + CT;
  const int oo = rid - ob_first;
  constexpr int C4 = (CT + 3) / 4;
  const OutLane<CT> ol(lane);
  constexpr int QA = OutLane<CT>::QA;

  const float beta1 = c.beta1, beta2 = c.beta2, eps = c.eps;
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  const uint32_t eps_safe = adam_eps_safe(eps);
  const bool sgd = a.solver == 1;
  int step_no = 0;
  uint32_t tg = 0;            // sub-tiles walked so far; every role counts the same sequence
  uint32_t staged = 0;        // sub-tiles whose row copies have been issued (first H warp)
  bool ok = true;


  if constexpr (RB) {  // 2 x 128 x 136 + 128 x 120 + 128 x 120 = 65,536 = 512 x 128
    if (role == 0) asm volatile("setmaxnreg.inc.sync.aligned.u32 136;");
    else if (role == 1) asm volatile("setmaxnreg.dec.sync.aligned.u32 120;");
    else asm volatile("setmaxnreg.dec.sync.aligned.u32 120;");
  }
#ifdef BBO_PHASE_TIMERS
  if (tid == 0) { for (int i = 0; i < 16; ++i) sh.t_wait[i >> 2][i & 3] = 0; sh.t_sort = 0; sh.t_adam[0] = sh.t_adam[1] = 0; }
  __syncthreads();
  const long long tt0_ = clock64();
#endif
  // Position in the schedule and per-step constants, the same for every role.
  struct StepInfo {
    int s0, Bs, T;
    float invB, aB;
    bool want_loss;
    uint32_t pprev;  // parity of the previous step's parameter barrier
  };
  // Traced steps (debug): the minibatch loss needs the row losses of every sub-tile and the
  // weights of before the update, so all roles meet here between the last sub-tile and the update.
  auto traced_loss = [&](const StepInfo& si) {
    __syncthreads();
    float sq = 0.f;
    for (int k = 0; k < d; ++k)
      for (int j = tid; j < H; j += nt) { const float w = W[L.oW1 + k * Hs + j]; sq = __fmaf_rn(w, w, sq); }
    for (int j = tid; j < H; j += nt)
      for (int o = 0; o < CT; ++o) { const float w = W[L.oW2 + o * L.WP + j]; sq = __fmaf_rn(w, w, sq); }
    for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
    if (lane == 0) sh.red[warp] = sq;
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
      for (int w = 0; w < (nt >> 5); ++w) tot += sh.red[w];
      float ls = 0.f;
      for (int b = 0; b < si.Bs; ++b) ls = __fadd_rn(ls, lossb[b]);
      const float loss = __fadd_rn(__fmul_rn(ls, si.invB), __fmul_rn(__fmul_rn(__fmul_rn(0.5f, c.alpha), si.invB), tot));
      a.trace[((size_t)config * a.K + fold) * a.trace_steps + step_no] = loss;
    }
    __syncthreads();
  };
  // Every role walks the same sequence of epochs, steps and sub-tiles; each gets its own copy of
  // the loops (the compiler then keeps only that role's state live inside them).
  auto walk = [&](auto&& on_epoch, auto&& on_step) {
    for (int e = 0; e < c.epochs; ++e) {
      __syncthreads();  // every role is through the previous epoch: row and activation buffers are idle
#ifdef BBO_PHASE_TIMERS
      const long long ts_ = clock64();
#endif
      build_epoch_order(keys, reinterpret_cast<uint32_t*>(sh.red), order, a.pi, n_tr, vb, holdout ? 0 : vs, a.seed, rng_config, rng_fold, e, tid, nt);
#ifdef BBO_PHASE_TIMERS
      if (tid == 0) sh.t_sort += clock64() - ts_;
#endif
      on_epoch();
      for (int s0 = 0; s0 < n_tr; s0 += B) {
        StepInfo si;
        si.s0 = s0;
        si.Bs = (n_tr - s0) < B ? (n_tr - s0) : B;
        si.T = (si.Bs + TB - 1) / TB;
        si.invB = __fdiv_rn(1.0f, (float)si.Bs);
        si.aB = __fmul_rn(c.alpha, si.invB);
        si.want_loss = a.trace != nullptr && step_no < a.trace_steps;
        si.pprev = (uint32_t)(step_no - 1) & 1u;
        on_step(si);
        tg += (uint32_t)si.T;
        ++step_no;
      }
    }
  };
  auto no_epoch_work = []() {};

  if (role == 1) {
    // ================= H: hidden layer of every sub-tile; its first warp stages the rows =================
    TileCursor pc{0, 0};  // staging cursor, one sub-tile ahead of the forward pass
    // one bulk copy per row, all landing on the buffer's barrier
    auto stage_tile = [&](const TileCursor& tc, uint32_t u) {
      const int nb = tc.rows(n_tr, B, TB);
      const uint32_t slot = u % kNX;
      BBO_ROLE_WAIT(3, ok = ok && role_wait(sh, &sh.xfree[slot], ((u / kNX) & 1u) ^ 1u));
      if (ok) {
        if (lane == 0) mbar_arrive_expect_tx(&sh.xfull[slot], (uint32_t)nb * row_bytes);
        __syncwarp();
        const uint16_t* rows = order + tc.s0 + tc.t0;
        for (int r = lane; r < nb; r += 32) bulk_copy_g2s(Xs + (slot * TB + r) * dp, a.X + (size_t)rows[r] * dp, row_bytes, &sh.xfull[slot]);
        staged = u + 1;
      }
    };
    walk([&]() {
      pc = TileCursor{0, 0};
      if (rw == 0) { stage_tile(pc, tg); pc.advance(n_tr, B, TB); }
    }, [&](const StepInfo& si) {
      const int Bs = si.Bs, T = si.T;
      const uint32_t pprev = si.pprev;
      if (step_no > 0) BBO_ROLE_WAIT(0, ok = ok && role_wait(sh, &sh.params, pprev));
      for (int t = 0; t < T; ++t) {
        const uint32_t u = tg + t;
        const int nb = (Bs - t * TB) < TB ? (Bs - t * TB) : TB;
        if (rw == 0 && pc.valid(n_tr)) { stage_tile(pc, u + 1); pc.advance(n_tr, B, TB); }
        BBO_ROLE_WAIT(1, ok = ok && role_wait(sh, &sh.xfull[u % kNX], (u / kNX) & 1u));
        BBO_ROLE_WAIT(2, ok = ok && role_wait(sh, &sh.a1free[u % kNA], ((u / kNA) & 1u) ^ 1u));
        if (ok) hidden_tiles(W, L, Xs + (u % kNX) * TB * dp, A1 + (u % kNA) * TB * L.WP, d, dp, Hs, nb, rid, hthreads);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.a1ready[u % kNA]);
      }
      if (si.want_loss) traced_loss(si);
    });
    if constexpr (RB) asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
  } else if (role == 2) {
    // ================= O: output layer, loss derivative =================
    double p1 = 1.0, p2 = 1.0;  // running beta^t (first lane of the role)
    walk(no_epoch_work, [&](const StepInfo& si) {
      const int s0 = si.s0, Bs = si.Bs, T = si.T;
      const float invB = si.invB;
      const bool want_loss = si.want_loss;
      const uint32_t pprev = si.pprev;
      if (rw == 0 && lane == 0) {
        p1 *= (double)beta1;
        p2 *= (double)beta2;
        sh.step[step_no & 1] = (float)((double)c.lr * sqrt(1.0 - p2) / (1.0 - p1));
      }
      if (step_no > 0) BBO_ROLE_WAIT(0, ok = ok && role_wait(sh, &sh.params, pprev));
      for (int t = 0; t < T; ++t) {
        const uint32_t u = tg + t;
        const int nb = (Bs - t * TB) < TB ? (Bs - t * TB) : TB;
        const uint16_t* rows = order + s0 + t * TB;
        BBO_ROLE_WAIT(1, ok = ok && role_wait(sh, &sh.a1ready[u % kNA], (u / kNA) & 1u));
        BBO_ROLE_WAIT(2, ok = ok && role_wait(sh, &sh.d2free[u % kND], ((u / kND) & 1u) ^ 1u));
        if (ok) {
          FitView vv;
          vv.W = W; vv.lossb = lossb;
          vv.A1 = A1 + (u % kNA) * TB * L.WP;
          vv.D2 = D2 + (u % kND) * TB * CS;
          for (int r0 = rw * 16; r0 < nb; r0 += a.nO * 16) {  // warp-uniform; a lane pair per row
            const int brow = r0 + (lane >> 1);
            const bool act = brow < nb;
            const float yv = act ? a.y[rows[brow]] : 0.f;  // labels / targets straight from global memory
            float z[QA];
            output_logits<CT>(vv, L, H, ol, act ? brow : nb - 1, z);
            row_delta<CT>(vv, a.task, CS, ol, z, yv, brow, act, invB, want_loss, t * TB + brow);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.d2ready[u % kND]);
      }
      if (want_loss) traced_loss(si);
    });
    if constexpr (RB) asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
  } else if (role == 3) {
    // ================= U: per hidden unit gW2, delta1, gb1; gb2 =================
    walk(no_epoch_work, [&](const StepInfo& si) {
      const int Bs = si.Bs, T = si.T;
      const float aB = si.aB;
      const bool want_loss = si.want_loss;
      float g2[UPT][CT], w2[UPT][CT], gb1[UPT], gb2 = 0.f;
#pragma unroll
      for (int un = 0; un < UPT; ++un) {
        gb1[un] = 0.f;
#pragma unroll
        for (int o = 0; o < CT; ++o) {
          g2[un][o] = 0.f;
          w2[un][o] = (role == 3 && uj + un < H) ? W[L.oW2 + o * L.WP + uj + un] : 0.f;
        }
      }
      for (int t = 0; t < T; ++t) {
        const uint32_t u = tg + t;
        const int nb = (Bs - t * TB) < TB ? (Bs - t * TB) : TB;
        BBO_ROLE_WAIT(1, ok = ok && role_wait(sh, &sh.d2ready[u % kND], (u / kND) & 1u));
        if (ok) {
          float* A1b = A1 + (u % kNA) * TB * L.WP;
          const float* D2b = D2 + (u % kND) * TB * CS;
          if (unit_any) {
            float* ap = A1b + uj;
#pragma unroll 2
            for (int b = 0; b < nb; ++b) {
              float av[UPT];
              if (UPT == 4) {
                const float4 tq = *reinterpret_cast<const float4*>(ap + b * L.WP);
                av[0] = tq.x; av[1 % UPT] = tq.y; av[2 % UPT] = tq.z; av[3 % UPT] = tq.w;
              } else {
                const float2 tq = *reinterpret_cast<const float2*>(ap + b * L.WP);
                av[0] = tq.x; av[1 % UPT] = tq.y;
              }
              float dl[C4 * 4];
#pragma unroll
              for (int o4 = 0; o4 < C4; ++o4) {
                const float4 tq = *reinterpret_cast<const float4*>(D2b + b * CS + 4 * o4);
                dl[4 * o4] = tq.x; dl[4 * o4 + 1] = tq.y; dl[4 * o4 + 2] = tq.z; dl[4 * o4 + 3] = tq.w;
              }
              float acc[UPT];
#pragma unroll
              for (int un = 0; un < UPT; ++un) acc[un] = 0.f;
#pragma unroll
              for (int o = 0; o < CT; ++o) {
#pragma unroll
                for (int un = 0; un < UPT; ++un) {
                  g2[un][o] = __fmaf_rn(av[un], dl[o], g2[un][o]);
                  acc[un] = __fmaf_rn(dl[o], w2[un][o], acc[un]);
                }
              }
              float d1[UPT];
#pragma unroll
              for (int un = 0; un < UPT; ++un) {
                d1[un] = av[un] > 0.f ? acc[un] : 0.f;
                gb1[un] = __fadd_rn(gb1[un], d1[un]);
              }
              if (UPT == 4) *reinterpret_cast<float4*>(ap + b * L.WP) = make_float4(d1[0], d1[1 % UPT], d1[2 % UPT], d1[3 % UPT]);
              else *reinterpret_cast<float2*>(ap + b * L.WP) = make_float2(d1[0], d1[1 % UPT]);
            }
          }
          if (o_role) for (int b = 0; b < nb; ++b) gb2 = __fadd_rn(gb2, D2b[b * CS + oo]);
        }
        __syncwarp();
        if (lane == 0) { mbar_arrive(&sh.d1ready[u % kNA]); mbar_arrive(&sh.d2free[u % kND]); }
      }
      if (want_loss) traced_loss(si);
      // ---- update of the W2 rows of this thread's units, their b1 entries, and b2 ----
      const float step = sh.step[step_no & 1];
      if (ok) {
#pragma unroll
        for (int un = 0; un < UPT; ++un) {
          const int j = uj + un;
          if (role == 3 && j < H) {
            float wu[CT + 1], mu[CT + 1], vu[CT + 1], gu[CT + 1];
#pragma unroll
            for (int o = 0; o < CT; ++o) {
              const int off = L.oW2 + o * L.WP + j;
              wu[o] = w2[un][o]; mu[o] = Msm[off]; vu[o] = Vsm[off];
              gu[o] = __fmaf_rn(aB, w2[un][o], g2[un][o]);
            }
            wu[CT] = W[L.ob1 + j]; mu[CT] = Msm[L.ob1 + j]; vu[CT] = Vsm[L.ob1 + j]; gu[CT] = gb1[un];
            if (sgd) {
              sgd_group<CT + 1>(wu, mu, gu, c.lr, beta1);
            } else if (!adam_group_fast<CT + 1>(wu, mu, vu, gu, beta1, beta2, omb1, omb2, step, eps, eps_safe)) {
#pragma unroll
              for (int o = 0; o < CT; ++o) wu[o] = w2[un][o];
              wu[CT] = W[L.ob1 + j];
              adam_params_ieee<CT + 1>(wu, mu, vu, step, eps);
            }
#pragma unroll
            for (int o = 0; o < CT; ++o) {
              const int off = L.oW2 + o * L.WP + j;
              W[off] = wu[o]; Msm[off] = mu[o]; Vsm[off] = vu[o];
            }
            W[L.ob1 + j] = wu[CT]; Msm[L.ob1 + j] = mu[CT]; Vsm[L.ob1 + j] = vu[CT];
          }
        }
        if (o_role) {
          const int off = L.ob2 + oo;
          if (sgd) {
            float w1[1] = {W[off]}, m1[1] = {Msm[off]};
            const float g1b[1] = {gb2};
            sgd_group<1>(w1, m1, g1b, c.lr, beta1);
            W[off] = w1[0]; Msm[off] = m1[0];
          } else {
            adam_one(W[off], Msm[off], Vsm[off], gb2, beta1, beta2, omb1, omb2, step, eps);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.params);
    });
    if constexpr (RB) asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
  } else {
    // ================= G: gradient tiles of W1, then L2 + Adam on them =================
    walk(no_epoch_work, [&](const StepInfo& si) {
      const int Bs = si.Bs, T = si.T;
      const float aB = si.aB;
      const bool want_loss = si.want_loss;
      float g1[8][8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) g1[i][j] = 0.f;
      for (int t = 0; t < T; ++t) {
        const uint32_t u = tg + t;
        const int nb = (Bs - t * TB) < TB ? (Bs - t * TB) : TB;
        BBO_ROLE_WAIT(1, ok = ok && role_wait(sh, &sh.d1ready[u % kNA], (u / kNA) & 1u));
        ok = ok && role_wait(sh, &sh.xfull[u % kNX], (u / kNX) & 1u);  // already complete: makes the copied rows visible here
        if (ok && has_tile) {
          const float* xp = Xs + (u % kNX) * TB * dp + k0;
          const float* da = A1 + (u % kNA) * TB * L.WP + jA;
          const float* db = A1 + (u % kNA) * TB * L.WP + jB;
          GradOperands opA, opB;
          opA.load(xp, da, db, 0, dp, L.WP);
          int b = 0;
#pragma unroll 1
          for (; b + 2 <= nb; b += 2) {
            opB.load(xp, da, db, b + 1, dp, L.WP);
            opA.accumulate(g1);
            opA.load(xp, da, db, b + 2 < nb ? b + 2 : b, dp, L.WP);
            opB.accumulate(g1);
          }
          if (b < nb) opA.accumulate(g1);
        }
        __syncwarp();
        if (lane == 0) { mbar_arrive(&sh.a1free[u % kNA]); mbar_arrive(&sh.xfree[u % kNX]); }
      }
      if (want_loss) traced_loss(si);
#ifdef BBO_PHASE_TIMERS
      const long long ta_ = clock64();
#endif
      const float step = sh.step[step_no & 1];
      // Every lane of the warp walks the eight tile rows (the tensor-memory accesses are
      // warp-wide); lanes without a tile, and rows k >= d, touch only their own moments.  The
      // moments of row i + 1 are requested before row i is updated.
      uint32_t mr[2][8], vr[2][8];
      tmem_load8_issue(tm, mr[0]);
      tmem_load8_issue(tm + 64u, vr[0]);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const bool live = ok && has_tile && (k0 + i) < d;
        const int offA = L.oW1 + (k0 + i) * Hs + jA, offB = L.oW1 + (k0 + i) * Hs + jB;
        float w8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (live) {
          const float4 wA = *reinterpret_cast<float4*>(W + offA), wB = *reinterpret_cast<float4*>(W + offB);
          w8[0] = wA.x; w8[1] = wA.y; w8[2] = wA.z; w8[3] = wA.w; w8[4] = wB.x; w8[5] = wB.y; w8[6] = wB.z; w8[7] = wB.w;
        }
        tmem_wait_loads(mr[i & 1], vr[i & 1]);
        if (i + 1 < 8) {
          tmem_load8_issue(tm + 8u * (i + 1), mr[(i + 1) & 1]);
          tmem_load8_issue(tm + 64u + 8u * (i + 1), vr[(i + 1) & 1]);
        }
        float m8[8], v8[8], g8[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          m8[j] = __uint_as_float(mr[i & 1][j]); v8[j] = __uint_as_float(vr[i & 1][j]);
          g8[j] = __fmaf_rn(aB, w8[j], g1[i][j]);
        }
        if (sgd) {
          sgd_group<8>(w8, m8, g8, c.lr, beta1);
        } else if (!adam_group_fast<8>(w8, m8, v8, g8, beta1, beta2, omb1, omb2, step, eps, eps_safe)) {
          // not certified: redo the parameter update from the stored weights with the IEEE routines
          if (live) {
            const float4 wA = *reinterpret_cast<float4*>(W + offA), wB = *reinterpret_cast<float4*>(W + offB);
            w8[0] = wA.x; w8[1] = wA.y; w8[2] = wA.z; w8[3] = wA.w; w8[4] = wB.x; w8[5] = wB.y; w8[6] = wB.z; w8[7] = wB.w;
          }
          adam_params_ieee<8>(w8, m8, v8, step, eps);
        }
        if (live) {
          *reinterpret_cast<float4*>(W + offA) = make_float4(w8[0], w8[1], w8[2], w8[3]);
          *reinterpret_cast<float4*>(W + offB) = make_float4(w8[4], w8[5], w8[6], w8[7]);
        }
        tmem_store8(tm + 8u * i, m8);
        tmem_store8(tm + 64u + 8u * i, v8);
      }
      tmem_wait_stores();
      __syncwarp();
#ifdef BBO_PHASE_TIMERS
      if (rw == 0 && lane == 0) sh.t_adam[0] += clock64() - ta_;
#endif
      if (lane == 0) mbar_arrive(&sh.params);
    });
    if constexpr (RB) asm volatile("setmaxnreg.dec.sync.aligned.u32 128;");
  }
  __syncthreads();

#ifdef BBO_PHASE_TIMERS
  if (tid == 0 && q == 0)
    printf("ROLES Hs=%d H=%d B=%d steps=%d tiles=%u | train %lld sort %lld adamG %lld | G wait params %lld d1ready %lld | H wait params %lld xfull %lld a1free %lld xfree %lld | O wait params %lld a1ready %lld d2free %lld | U wait d2ready %lld\n",
           Hs, H, B, step_no, tg, clock64() - tt0_, sh.t_sort, sh.t_adam[0], sh.t_wait[0][0], sh.t_wait[0][1], sh.t_wait[1][0], sh.t_wait[1][1], sh.t_wait[1][2], sh.t_wait[1][3], sh.t_wait[2][0], sh.t_wait[2][1], sh.t_wait[2][2], sh.t_wait[3][1]);
#endif
  // ---- held-out score: the same hidden and output code, block-phased, on the held-out rows ----
  if (tid == 0) { sh.correct = 0; sh.sq = 0.f; }
  __syncthreads();
  const int n_warps = nt >> 5;
  for (int t0 = 0; t0 < vs; t0 += TB) {
    const int nb = (vs - t0) < TB ? (vs - t0) : TB;
    {
      const int vec = dp >> 2;
      const float* src = holdout ? a.Xt : a.X;
      for (int i = tid; i < nb * vec; i += nt) {
        const int r = i / vec, qv = i - r * vec;
        const int row = holdout ? t0 + r : a.pi[vb + t0 + r];
        reinterpret_cast<float4*>(Xs)[i] = reinterpret_cast<const float4*>(src + (size_t)row * dp)[qv];
      }
    }
    __syncthreads();
    hidden_tiles(W, L, Xs, A1, d, dp, Hs, nb, tid, nt);
    __syncthreads();
    for (int r0 = warp * 32; r0 < nb; r0 += n_warps * 32) {  // warp-uniform
      const int brow = r0 + lane;
      if (brow < nb) {
        const float yv = holdout ? a.yt[t0 + brow] : a.y[a.pi[vb + t0 + brow]];
        float z[CT];
        row_logits<CT>(W, L, H, A1 + brow * L.WP, z);
        if (a.task == 0 && a.metric == 1) {
          // negative log-likelihood of the true class
          float mx, sum, ex[CT];
          row_softmax<CT>(z, mx, ex, sum);
          const int label = (int)yv;
          float zl = 0.f;
#pragma unroll
          for (int o = 0; o < CT; ++o) if (o == label) zl = z[o];
          D2[brow * CS] = __fsub_rn(logf(sum), __fsub_rn(zl, mx));
        } else if (a.task == 0) {
          // prediction: lowest index attaining the maximum (ascending scan with strict >)
          float best = z[0];
          int besti = 0;
#pragma unroll
          for (int o = 1; o < CT; ++o) if (z[o] > best) { best = z[o]; besti = o; }
          if (besti == (int)yv) atomicAdd(&sh.correct, 1);
        } else {
          D2[brow * CS] = __fsub_rn(z[0], yv);
        }
      }
    }
    __syncthreads();
    if ((a.task != 0 || a.metric == 1) && tid == 0) {  // row sums in ascending row order
      float sq = sh.sq;
      if (a.metric == 1) for (int b = 0; b < nb; ++b) sq = __fadd_rn(sq, fabsf(D2[b * CS]));
      else for (int b = 0; b < nb; ++b) { const float r = D2[b * CS]; sq = __fmaf_rn(r, r, sq); }
      sh.sq = sq;
    }
    __syncthreads();
  }
  if (tid == 0) {
    float score;
    if (a.task == 0 && a.metric == 0) {
      score = __fdiv_rn((float)sh.correct, (float)vs);
    } else {
      score = -__fdiv_rn(sh.sq, (float)vs);
      if (score != score) score = __int_as_float(0xFF800000);
    }
    if (sh.abort) {  // a wait ran out: the fit is void, and the host reports the time-out
      score = __int_as_float(0x7FC00000);
      atomicExch(a.status, 1);
    }
    a.fold_scores[(size_t)config * a.K + fold] = score;
  }
  if (a.keep_theta != nullptr && config == a.n_configs - 1 && fold == a.K - 1) {
    const int n1 = d * H, n2 = H * CT;
    for (int i = tid; i < n1; i += nt) a.keep_theta[i] = W[L.oW1 + (i / H) * Hs + (i % H)];
    for (int i = tid; i < H; i += nt) a.keep_theta[n1 + i] = W[L.ob1 + i];
    for (int i = tid; i < n2; i += nt) a.keep_theta[n1 + H + i] = W[L.oW2 + (i % CT) * L.WP + (i / CT)];
    for (int i = tid; i < CT; i += nt) a.keep_theta[n1 + H + n2 + i] = W[L.ob2 + i];
  }
  // a fit that gave up may still have row copies in flight: give them a bounded time to land
  // before the shared memory is handed back
  if (sh.abort && role == 1 && rw == 0 && lane == 0) {
    for (uint32_t u = staged > (uint32_t)kNX ? staged - kNX : 0u; u < staged; ++u)
      for (int i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(&sh.xfull[u % kNX], (u / kNX) & 1u)) break;
  }
  tmem_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(sh.tmem_base, (uint32_t)a.tmem_cols);
}

// One CTA per fit; blockIdx.x indexes this launch's fit list (costliest first).
template <int CT, int HSC, int DPC, int NTMAX, int MINB, bool RB>
__global__ void __launch_bounds__(NTMAX, MINB) mlp_cv_fit_roles_kernel(const FitArgs a) {
  extern __shared__ __align__(128) float smem_roles[];
  __shared__ RoleShared sh;
  run_fit_roles<CT, HSC, DPC, RB>(a, blockIdx.x, smem_roles, sh);
}

}  // namespace bbo
