// One CTA trains and scores one (configuration, fold) fit with the parameters and the Adam
// moments resident on chip (paper sec. 2: the function evaluated is the cross-validation
// score of a model on a dataset; Table 1: MLP-adam, metrics acc / mse; sec. 5: the model
// evaluation is what runs on the GPU, with the data kept there).
//
// Arithmetic contract.  Every accumulation runs in one fixed order, so results do not
// depend on the thread mapping: forward sums ascend over the input index with fused
// multiply-adds starting from the bias; gradient sums ascend over the minibatch row starting
// from zero; the softmax uses the explicit exponential of device_math.cuh and sums its
// denominator in ascending class order; division and square root are IEEE; the Adam
// bias-correction products are kept in binary64 and the step size is rounded to binary32
// once per step.  Threads own outputs, never partial sums: there is no split reduction
// anywhere on the training path.
//
// Work decomposition per minibatch, in sub-tiles of TB rows (H padded to Hs = 8*ceil(H/8),
// d padded to dp = 8*ceil(d/8)); about Hs threads per fit, few and register-heavy, because
// shared-memory instruction issue, not capacity, is what limits the register-tiled loops:
//   stage   cp.async gather of the next sub-tile's rows, double buffered
//   hidden  8x4 register tiles of A1 = relu(X W1 + b1), k ascending
//   output  a lane pair per row, each lane half of the classes; W2 is kept class-major so one
//           16-byte load feeds four steps of a chain; operands fetched one iteration ahead;
//           softmax and loss derivative in the same lanes (two shuffles per scan)
//   unit    one thread per hidden unit j: gW2[j][:], delta1[:, j] (in place over A1), gb1[j]
//   gW1     8x8 register tiles that persist across sub-tiles, b ascending; the owner applies
//           the L2 term and Adam to exactly its elements.  The first and second moments of W1
//           live in tensor memory: each owner thread stores and reloads its own 128 words once
//           per step (tcgen05.st / tcgen05.ld), which leaves shared memory to the parameters
//           and the buffers and lets several fits share an SM
// HSC / DPC: compile-time Hs / dp (0 = taken from the arguments) so that every shared-memory
// access of the hot loops is base + immediate.
#pragma once
#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

#include "device_math.cuh"
#include "fit_common.cuh"
#include "sm100_primitives.cuh"

// Optional phase timers (compile with -DBBO_PHASE_TIMERS): thread 0 accumulates clock64 deltas
// per phase, as seen after the barrier that ends the phase, and block 0 of each launch prints
// them.  Compiled out by default.
#ifdef BBO_PHASE_TIMERS
#include <cstdio>
#define BBO_PHASE_BEGIN() long long ph_t_ = clock64()
#define BBO_PHASE(i) do { if (tid == 0) { const long long t_ = clock64(); sh.phase[i] += t_ - ph_t_; ph_t_ = t_; } } while (0)
#else
#define BBO_PHASE_BEGIN() do { } while (0)
#define BBO_PHASE(i) do { } while (0)
#endif

namespace bbo {

struct FitView {  // per-fit pointers into shared memory
  float *W, *M, *V;     // M, V hold the moments of b1, W2, b2 only and are biased: M[off], V[off] are valid for off >= ob1
  uint16_t* order;
  float *lossb, *ys, *D2, *Xs, *A1;
  uint64_t* keys;
};

// Asynchronous gather of nb dataset rows into buffer `buf` of Xs / ys.  Rows nb..TB-1 are
// zero-filled so that the forward tiles read defined values.  row_of(r) = dataset row.
template <typename RowFn>
__device__ __forceinline__ void stage_rows_async(const FitArgs& a, const float* Xsrc, const float* ysrc, const FitView& v,
                                                 int dp, int buf, int nb, RowFn row_of, int tid, int nt) {
  const int vec = dp >> 2;
  float* xs = v.Xs + buf * a.TB * dp;
  for (int i = tid; i < a.TB * vec; i += nt) {
    const int r = i / vec, q = i - r * vec;
    float4* dst = reinterpret_cast<float4*>(xs) + i;
    if (r < nb) cp_async_16(dst, reinterpret_cast<const float4*>(Xsrc + (size_t)row_of(r) * dp) + q);
    else *dst = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int r = tid; r < nb; r += nt) cp_async_4(v.ys + buf * a.TB + r, ysrc + row_of(r));
  cp_async_commit();
}

__device__ __forceinline__ float f4_get(const float4& v, int i) {
  return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// A1 = relu(Xs W1 + b1) for the sub-tile; each thread owns R rows x 4 columns, k ascending.
template <int R>
__device__ __forceinline__ void forward_tiles(const FitView& v, const Layout& L, const float* xs, int d, int dp,
                                              int Hs, int nb, int tid, int nt) {
  const int JG = Hs >> 2, n_tiles = ((nb + R - 1) / R) * JG;
  const int d4 = d >> 2;
  for (int t = tid; t < n_tiles; t += nt) {
    const int bg = t / JG, jg = t - bg * JG;
    const int b0 = bg * R, j0 = jg << 2;
    const float4 bias = *reinterpret_cast<const float4*>(v.W + L.ob1 + j0);
    float acc[R][4];
#pragma unroll
    for (int i = 0; i < R; ++i) { acc[i][0] = bias.x; acc[i][1] = bias.y; acc[i][2] = bias.z; acc[i][3] = bias.w; }
    const float* xrow = xs + b0 * dp;
    const float* wp = v.W + L.oW1 + j0;
#pragma unroll 2
    for (int k4 = 0; k4 < d4; ++k4) {
      float4 xv[R];
#pragma unroll
      for (int i = 0; i < R; ++i) xv[i] = *reinterpret_cast<const float4*>(xrow + i * dp + 4 * k4);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 w = *reinterpret_cast<const float4*>(wp + (4 * k4 + kk) * Hs);
#pragma unroll
        for (int i = 0; i < R; ++i) {
          const float x = f4_get(xv[i], kk);
          acc[i][0] = __fmaf_rn(x, w.x, acc[i][0]);
          acc[i][1] = __fmaf_rn(x, w.y, acc[i][1]);
          acc[i][2] = __fmaf_rn(x, w.z, acc[i][2]);
          acc[i][3] = __fmaf_rn(x, w.w, acc[i][3]);
        }
      }
    }
    for (int k = d4 << 2; k < d; ++k) {
      const float4 w = *reinterpret_cast<const float4*>(wp + k * Hs);
#pragma unroll
      for (int i = 0; i < R; ++i) {
        const float x = xrow[i * dp + k];
        acc[i][0] = __fmaf_rn(x, w.x, acc[i][0]);
        acc[i][1] = __fmaf_rn(x, w.y, acc[i][1]);
        acc[i][2] = __fmaf_rn(x, w.z, acc[i][2]);
        acc[i][3] = __fmaf_rn(x, w.w, acc[i][3]);
      }
    }
#pragma unroll
    for (int i = 0; i < R; ++i) {
      float4 o;
      o.x = acc[i][0] > 0.f ? acc[i][0] : 0.f;
      o.y = acc[i][1] > 0.f ? acc[i][1] : 0.f;
      o.z = acc[i][2] > 0.f ? acc[i][2] : 0.f;
      o.w = acc[i][3] > 0.f ? acc[i][3] : 0.f;
      *reinterpret_cast<float4*>(v.A1 + (b0 + i) * L.WP + j0) = o;
    }
  }
}

// Sub-tiles of at most 16 rows (small minibatches, ragged ends) take 4-row tiles so that all
// threads share the work; full sub-tiles take 8-row tiles (fewer loads per multiply-add).
// LEAN kernels (register-capped, see mlp_cv_fit_kernel) always take 4-row tiles: the 8-row tile
// does not fit beside the gradient tile in their registers.
template <bool LEAN>
__device__ __forceinline__ void forward_hidden(const FitView& v, const Layout& L, const float* xs, int d, int dp,
                                               int Hs, int nb, int tid, int nt) {
  if (LEAN || nb <= 16) forward_tiles<4>(v, L, xs, d, dp, Hs, nb, tid, nt);
  else forward_tiles<8>(v, L, xs, d, dp, Hs, nb, tid, nt);
}

// Output layer.  A lane owns one row of the sub-tile and one half of the classes: classes
// [0, QA) for the even lane of a pair, [QA, CT) for the odd lane, QA = ceil(CT / 2).  One
// 16-byte load of the A1 row and one of each class row of W2 feed four steps of every chain:
// z2[b][o] = b2[o] + sum_j A1[b][j] W2[j][o], j ascending.  (Shared-memory loads are what
// bounds this phase, and this shape needs the fewest of them per multiply-add.)
template <int CT>
struct OutLane {
  static constexpr int QA = (CT + 1) / 2, QB = CT - QA;
  int half, o0, nq;  // this lane's classes are o0 .. o0 + nq - 1
  __device__ __forceinline__ explicit OutLane(int lane) {
    half = lane & 1;
    o0 = half ? QA : 0;
    nq = half ? QB : QA;
  }
  __device__ __forceinline__ int cls(int q) const { return q < nq ? o0 + q : o0 + (nq > 0 ? nq - 1 : -o0); }
};

template <int CT>
__device__ __forceinline__ void output_logits(const FitView& v, const Layout& L, int H, const OutLane<CT>& ol, int row,
                                              float (&z)[OutLane<CT>::QA]) {
  constexpr int QA = OutLane<CT>::QA;
  const float* wrow[QA];
#pragma unroll
  for (int q = 0; q < QA; ++q) {
    const int o = ol.cls(q);  // lanes with fewer classes repeat their last one (result unused)
    z[q] = v.W[L.ob2 + o];
    wrow[q] = v.W + L.oW2 + o * L.WP;
  }
  const float* arow = v.A1 + row * L.WP;
  // Few warps run this phase, so nothing else hides the load latency: the operands of the
  // next four steps are fetched before the current four multiply-adds are issued.
  int j = 0;
  float4 a_nx = *reinterpret_cast<const float4*>(arow);
  float4 w_nx[QA];
#pragma unroll
  for (int q = 0; q < QA; ++q) w_nx[q] = *reinterpret_cast<const float4*>(wrow[q]);
#pragma unroll 2
  for (; j + 4 <= H; j += 4) {
    const float4 a = a_nx;
    float4 w[QA];
#pragma unroll
    for (int q = 0; q < QA; ++q) w[q] = w_nx[q];
    // rows are padded by four floats, so the read past the last step stays inside the row
    a_nx = *reinterpret_cast<const float4*>(arow + j + 4);
#pragma unroll
    for (int q = 0; q < QA; ++q) w_nx[q] = *reinterpret_cast<const float4*>(wrow[q] + j + 4);
#pragma unroll
    for (int q = 0; q < QA; ++q) z[q] = __fmaf_rn(a.x, w[q].x, z[q]);
#pragma unroll
    for (int q = 0; q < QA; ++q) z[q] = __fmaf_rn(a.y, w[q].y, z[q]);
#pragma unroll
    for (int q = 0; q < QA; ++q) z[q] = __fmaf_rn(a.z, w[q].z, z[q]);
#pragma unroll
    for (int q = 0; q < QA; ++q) z[q] = __fmaf_rn(a.w, w[q].w, z[q]);
  }
  for (; j < H; ++j) {
    const float a = arow[j];
#pragma unroll
    for (int q = 0; q < QA; ++q) z[q] = __fmaf_rn(a, wrow[q][j], z[q]);
  }
}

// Adam on N parameters held in registers, first pass: moments updated in place, parameters
// updated with the branch-free ratio.  Returns 1 when every ratio was computed inside the range
// in which it equals the IEEE result; otherwise the caller discards th[] and redoes the
// parameter update with adam_params_ieee from the updated moments.
template <int N>
__device__ __forceinline__ uint32_t adam_group_fast(float (&th)[N], float (&m)[N], float (&vv)[N], const float (&g)[N],
                                                    float beta1, float beta2, float omb1, float omb2, float step,
                                                    float eps, uint32_t eps_safe) {
  AdamCert cert;
#pragma unroll
  for (int e = 0; e < N; ++e) {
    m[e] = __fmaf_rn(beta1, m[e], __fmul_rn(omb1, g[e]));
    vv[e] = __fmaf_rn(beta2, vv[e], __fmul_rn(__fmul_rn(omb2, g[e]), g[e]));
    th[e] = __fsub_rn(th[e], __fmul_rn(step, adam_ratio_fast(m[e], vv[e], eps, cert)));
  }
  return eps_safe & cert.ok();
}

// Second pass for a group the first pass could not certify: IEEE square root and division.
// A NaN moment gives NaN either way, and skipping the library call there keeps fits whose
// parameters have become NaN at full speed.
template <int N>
__device__ __forceinline__ void adam_params_ieee(float (&th)[N], const float (&m)[N], const float (&vv)[N], float step,
                                                 float eps) {
#pragma unroll
  for (int e = 0; e < N; ++e) {
    float q;
    if (m[e] != m[e] || vv[e] != vv[e]) q = __fadd_rn(m[e], vv[e]);
    else q = adam_ratio_ieee(m[e], vv[e], eps);
    th[e] = __fsub_rn(th[e], __fmul_rn(step, q));
  }
}

// Momentum SGD with Nesterov look-ahead on N parameters held in registers (vel: the velocity,
// kept where Adam keeps its first moments): vel = momentum vel - lr g;
// theta += momentum vel - lr g with the new velocity; lr g rounded once.
template <int N>
__device__ __forceinline__ void sgd_group(float (&th)[N], float (&vel)[N], const float (&g)[N], float lr,
                                          float momentum) {
#pragma unroll
  for (int e = 0; e < N; ++e) {
    const float t = __fmul_rn(lr, g[e]);
    vel[e] = __fmaf_rn(momentum, vel[e], -t);
    th[e] = __fadd_rn(th[e], __fmaf_rn(momentum, vel[e], -t));
  }
}

// Operands of one row of the W1 gradient tile: x[b][k0..k0+7] and delta1[b][jA..jA+3, jB..jB+3].
struct GradOperands {
  float4 x0, x1, dA, dB;
  __device__ __forceinline__ void load(const float* xp, const float* da, const float* db, int b, int dp, int wp) {
    x0 = *reinterpret_cast<const float4*>(xp + b * dp);
    x1 = *reinterpret_cast<const float4*>(xp + b * dp + 4);
    dA = *reinterpret_cast<const float4*>(da + b * wp);
    dB = *reinterpret_cast<const float4*>(db + b * wp);
  }
  __device__ __forceinline__ void accumulate(float (&g1)[8][8]) const {
    const float xk[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
    const float ds[8] = {dA.x, dA.y, dA.z, dA.w, dB.x, dB.y, dB.z, dB.w};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) g1[i][j] = __fmaf_rn(xk[i], ds[j], g1[i][j]);
  }
};

struct BlockShared {  // block-wide scalars
  float step[2];  // Adam step size, indexed by step parity (writer runs ahead of readers)
  int correct;
  float sq;
  float red[32];
  uint32_t tmem_base;  // tensor-memory allocation of the CTA
#ifdef BBO_PHASE_TIMERS
  long long phase[12];
#endif
};

// Softmax statistics of one row from the logits held by a lane pair: the running maximum and
// the denominator are taken over the classes in ascending order; the odd lane continues both
// scans from the even lane's result, and both lanes end up with the row's values.  All 32 lanes
// must call it.
template <int CT>
__device__ __forceinline__ void softmax_scan(const OutLane<CT>& ol, const float (&z)[OutLane<CT>::QA], float& mx,
                                             float (&ex)[OutLane<CT>::QA], float& sum) {
  constexpr int QA = OutLane<CT>::QA;
  const int lane = threadIdx.x & 31;
  // maximum: ascending scan with strict >, started by the even lane
  mx = z[0];
#pragma unroll
  for (int q = 1; q < QA; ++q) if (z[q] > mx) mx = z[q];
  const float m_even = __shfl_sync(0xffffffffu, mx, lane & ~1);
  if (ol.half) {
    mx = m_even;
#pragma unroll
    for (int q = 0; q < QA; ++q) if (q < ol.nq && z[q] > mx) mx = z[q];
  }
  mx = __shfl_sync(0xffffffffu, mx, lane | 1);
#pragma unroll
  for (int q = 0; q < QA; ++q) ex[q] = spec_expf(__fsub_rn(z[q], mx));
  // denominator: ascending sum from zero, continued by the odd lane
  sum = 0.f;
  if (!ol.half) {
#pragma unroll
    for (int q = 0; q < QA; ++q) sum = __fadd_rn(sum, ex[q]);
  }
  const float s_even = __shfl_sync(0xffffffffu, sum, lane & ~1);
  if (ol.half) {
    sum = s_even;
#pragma unroll
    for (int q = 0; q < QA; ++q) if (q < ol.nq) sum = __fadd_rn(sum, ex[q]);
  }
  sum = __shfl_sync(0xffffffffu, sum, lane | 1);
}

// Loss derivative of one row from the logits held by a lane pair, written to D2[row][:].
// All 32 lanes must call it; `active` gates the stores.
template <int CT>
__device__ __forceinline__ void row_delta(const FitView& v, int task, int CS, const OutLane<CT>& ol,
                                          const float (&z)[OutLane<CT>::QA], float yv, int row, bool active, float invB,
                                          bool want_loss, int loss_idx) {
  constexpr int QA = OutLane<CT>::QA;
  if (task == 0) {
    const int label = (int)yv;
    float mx, sum, ex[QA];
    softmax_scan<CT>(ol, z, mx, ex, sum);
    // probabilities: branch-free division first; the IEEE routine only where it cannot be certified
    float pr[QA];
    uint32_t safe = 1u;
#pragma unroll
    for (int q = 0; q < QA; ++q) pr[q] = softmax_ratio_fast(ex[q], sum, safe);
    if (!safe) {
#pragma unroll
      for (int q = 0; q < QA; ++q) pr[q] = sum != sum ? sum : __fdiv_rn(ex[q], sum);  // NaN row: skip the library's special cases
    }
    float zl = 0.f;
#pragma unroll
    for (int q = 0; q < QA; ++q) {
      const int o = ol.o0 + q;
      if (active && q < ol.nq) v.D2[row * CS + o] = __fmul_rn(__fsub_rn(pr[q], o == label ? 1.0f : 0.0f), invB);
      if (o == label) zl = z[q];
    }
    if (want_loss && active && label >= ol.o0 && label < ol.o0 + ol.nq)
      v.lossb[loss_idx] = __fsub_rn(logf(sum), __fsub_rn(zl, mx));
    return;
  }
  if (active && !ol.half) {
    const float r = __fsub_rn(z[0], yv);
    if (want_loss) v.lossb[loss_idx] = __fmul_rn(__fmul_rn(0.5f, r), r);
    v.D2[row * CS] = __fmul_rn(r, invB);
  }
}

// The whole fit.  CT: class count.  PL: pipelined schedule (extra warps for the output layer).
// LEAN: the kernel is built for fewer registers per thread than its tiles like (smaller forward
// tile, one operand set in the gradient loop); results are the same bit for bit.
template <int CT, int HSC, int DPC, bool PL, bool LEAN>
__device__ __forceinline__ void run_fit(const FitArgs& a, int q, float* smem, BlockShared& sh) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, n_warps = nt >> 5;
  const int2 cf = a.fits[q];
  const int config = cf.x, fold = cf.y;
  const uint32_t rng_config = a.config_keys ? (uint32_t)a.config_keys[config] : (uint32_t)(config + a.config_base);  // keys the random streams
  const Config c = a.configs[config];
  const int H = c.hidden, d = a.d, CS = a.CS, TB = a.TB;
  const int dp = DPC ? DPC : a.dp;
  const int Hs = HSC ? HSC : a.Hs;
  const Layout L(d, Hs, CT, CS);
  // Hold-out mode (paper sec. 6.2: the generalisation score comes from rows kept out of the
  // optimisation): every row trains, in the order of the fold permutation, and the score is taken
  // on the rows of a second matrix; the fold index then only keys the random streams.
  const bool holdout = a.Xt != nullptr;
  const uint32_t rng_fold = holdout ? kHoldoutFoldKey : (uint32_t)fold;
  int vb = 0, vs = 0;
  if (!holdout) fold_segment(a.n, a.K, fold, &vb, &vs);
  const int n_tr = a.n - vs;
  if (holdout) vs = a.n_test;  // rows to score
  const int B = c.batch_size < n_tr ? c.batch_size : n_tr;

#ifdef BBO_PHASE_TIMERS
  if (tid < 12) sh.phase[tid] = 0;
#endif
  BBO_PHASE_BEGIN();
  FitView v;
  v.W = smem;
  v.M = v.W + L.PS - L.ob1;
  v.V = v.M + L.PT;
  char* p = reinterpret_cast<char*>(v.W + L.PS + 2 * L.PT);
  v.order = reinterpret_cast<uint16_t*>(p); p += a.order_bytes;
  v.lossb = reinterpret_cast<float*>(p);    p += round_up(4 * a.loss_cap, 16);
  v.ys = reinterpret_cast<float*>(p);       p += (PL ? 12 : 8) * TB;   // one label buffer per row buffer
  v.D2 = reinterpret_cast<float*>(p);       p += 4 * TB * CS;
  v.Xs = reinterpret_cast<float*>(p);
  v.A1 = v.Xs + (PL ? 3 : 2) * TB * dp;                                 // PL: three row buffers, two of A1
  v.keys = reinterpret_cast<uint64_t*>(p);

  // ---- initialisation: Glorot-uniform parameters, zero moments ----
  for (int i = tid; i < L.PS + 2 * L.PT; i += nt) v.W[i] = 0.f;
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
        if (idx < n1) { const int k = idx / H, j = idx - k * H; v.W[L.oW1 + k * Hs + j] = glorot_value(word_of(r, w), bound1); }
      }
    }
    for (int blk = tid; blk < ((H + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 1u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int j = 4 * blk + w; if (j < H) v.W[L.ob1 + j] = glorot_value(word_of(r, w), bound1); }
    }
    for (int blk = tid; blk < ((n2 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 2u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n2) { const int j = idx / CT, o = idx - j * CT; v.W[L.oW2 + o * L.WP + j] = glorot_value(word_of(r, w), bound2); }
      }
    }
    for (int blk = tid; blk < ((CT + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, rng_config, rng_fold, 3u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int o = 4 * blk + w; if (o < CT) v.W[L.ob2 + o] = glorot_value(word_of(r, w), bound2); }
    }
  }
  __syncthreads();

  BBO_PHASE(0);
  // ---- thread roles ----
  const int KG = dp >> 3, JG8 = Hs >> 3;
  const bool has_tile = tid < KG * JG8;            // gW1 tile owner (host guarantees KG*JG8 <= nt)
  const int kg = has_tile ? tid / JG8 : 0, jg = has_tile ? tid - kg * JG8 : 0;
  const int k0 = kg << 3, jA = jg << 2, jB = (jg + JG8) << 2;
  // Tensor-memory home of this thread's W1 moments.  A warp reaches the 32 lanes of its quarter
  // (warp index mod 4); every group of four tile-owner warps gets 128 columns: first moments of
  // tile row i in columns 8 i .. 8 i + 7, second moments in 64 + 8 i ..
  const bool tile_warp = warp < ((KG * JG8 + 31) >> 5);
  const uint32_t tm = sh.tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + 128u * (uint32_t)(warp >> 2);
  if (tile_warp) {
    float zero16[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) zero16[i] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tmem_store16(tm + 16u * i, zero16);
    tmem_wait_stores();
  }
  const bool unit_role = tid < H;                   // hidden unit tid: W2 column, b1, delta1 column
  const int o_first = nt >= 64 ? nt - 32 : 0;       // gb2 / b2 owners sit in the last warp, away from the unit threads
  const bool o_role = tid >= o_first && tid < o_first + CT;
  const int oo = tid - o_first;
  const int nt_main = PL ? nt - 32 * a.extra_warps : nt;  // PL: the last warps only run the output layer
  const int out_w0 = nt_main >> 5;
  const OutLane<CT> ol(lane);                       // output phase: lane pair = one row, each lane half the classes
  constexpr int QA = OutLane<CT>::QA;

  const float beta1 = c.beta1, beta2 = c.beta2, eps = c.eps;
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  const uint32_t eps_safe = adam_eps_safe(eps);
  double p1 = 1.0, p2 = 1.0;  // running beta^t (thread 0 only)
  int step_no = 0;

  for (int e = 0; e < c.epochs; ++e) {
    build_epoch_order(v.keys, reinterpret_cast<uint32_t*>(sh.red), v.order, a.pi, n_tr, vb, holdout ? 0 : vs, a.seed, rng_config, rng_fold, e, tid, nt);
    BBO_PHASE(1);
    int buf = 0, abuf = 0;
    {  // first sub-tile of the epoch
      const int Bs0 = n_tr < B ? n_tr : B, nb0 = Bs0 < TB ? Bs0 : TB;
      const uint16_t* rows = v.order;
      stage_rows_async(a, a.X, a.y, v, dp, 0, nb0, [&](int r) { return (int)rows[r]; }, tid, nt);
    }
    for (int s0 = 0; s0 < n_tr; s0 += B) {
      const int Bs = (n_tr - s0) < B ? (n_tr - s0) : B;
      const float invB = __fdiv_rn(1.0f, (float)Bs);
      const float aB = __fmul_rn(c.alpha, invB);
      const bool want_loss = a.trace != nullptr && step_no < a.trace_steps;
      if (tid == 0) {
        p1 *= (double)beta1;
        p2 *= (double)beta2;
        sh.step[step_no & 1] = (float)((double)c.lr * sqrt(1.0 - p2) / (1.0 - p1));
      }
      float g1[8][8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) g1[i][j] = 0.f;
      float g2[CT], w2[CT], gb1 = 0.f, gb2 = 0.f;
#pragma unroll
      for (int o = 0; o < CT; ++o) { g2[o] = 0.f; w2[o] = unit_role ? v.W[L.oW2 + o * L.WP + tid] : 0.f; }

      // ---- the phases of one sub-tile; A1b: the sub-tile's buffer of hidden activations ----
      // output layer, softmax / residual, loss derivative (lane pairs own rows), by warps w0 .. w0+nw-1
      auto output_phase = [&](float* A1b, const float* ysb, int nb, int t0, int w0, int nw) {
        FitView vv = v;
        vv.A1 = A1b;
        for (int r0 = (warp - w0) * 16; r0 < nb; r0 += nw * 16) {  // warp-uniform
          const int brow = r0 + (lane >> 1);
          const bool act = brow < nb;
          float z[QA];
          output_logits<CT>(vv, L, H, ol, act ? brow : nb - 1, z);
          row_delta<CT>(vv, a.task, CS, ol, z, act ? ysb[brow] : 0.f, brow, act, invB, want_loss, t0 + brow);
        }
      };
      // hidden unit tid: gW2[tid][:], delta1[:, tid] in place over A1, gb1[tid]; b ascending
      auto unit_phase = [&](float* A1b, int nb) {
        if (unit_role) {
          float* ap = A1b + tid;
          constexpr int C4 = (CT + 3) / 4;
          int b = 0;
          for (; b + 4 <= nb; b += 4) {  // four rows at a time: loads first, then four independent delta1 chains
            float a1r[4], dl[4][C4 * 4], acc[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              a1r[r] = ap[(b + r) * L.WP];
#pragma unroll
              for (int o4 = 0; o4 < C4; ++o4) {
                const float4 t = *reinterpret_cast<const float4*>(v.D2 + (b + r) * CS + 4 * o4);
                dl[r][4 * o4] = t.x; dl[r][4 * o4 + 1] = t.y; dl[r][4 * o4 + 2] = t.z; dl[r][4 * o4 + 3] = t.w;
              }
              acc[r] = 0.f;
            }
#pragma unroll
            for (int o = 0; o < CT; ++o) {
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                g2[o] = __fmaf_rn(a1r[r], dl[r][o], g2[o]);
                acc[r] = __fmaf_rn(dl[r][o], w2[o], acc[r]);
              }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const float d1 = a1r[r] > 0.f ? acc[r] : 0.f;
              ap[(b + r) * L.WP] = d1;
              gb1 = __fadd_rn(gb1, d1);
            }
          }
          for (; b < nb; ++b) {
            const float a1 = ap[b * L.WP];
            float acc = 0.f;
#pragma unroll
            for (int o = 0; o < CT; ++o) {
              const float dv = v.D2[b * CS + o];
              g2[o] = __fmaf_rn(a1, dv, g2[o]);
              acc = __fmaf_rn(dv, w2[o], acc);
            }
            const float d1 = a1 > 0.f ? acc : 0.f;
            ap[b * L.WP] = d1;
            gb1 = __fadd_rn(gb1, d1);
          }
        }
        if (o_role) for (int b = 0; b < nb; ++b) gb2 = __fadd_rn(gb2, v.D2[b * CS + oo]);
      };
      // gW1 tile: rows k0..k0+7, columns jA..jA+3 and jB..jB+3, b ascending
      auto gw1_phase = [&](const float* xs, const float* A1b, int nb) {
        if (has_tile) {
          const float* xp = xs + k0;
          const float* da = A1b + jA;
          const float* db = A1b + jB;
          if constexpr (LEAN) {
            GradOperands op;
#pragma unroll 1
            for (int b = 0; b < nb; ++b) {
              op.load(xp, da, db, b, dp, L.WP);
              op.accumulate(g1);
            }
          } else {
            // Two operand sets in flight: the loads of row b + 1 are issued before the multiply-adds
            // of row b, so a warp does not sit out the shared-memory latency once per row.
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
        }
      };
      // prefetch of the sub-tile that follows (t0 of step s0) in this epoch into row buffer `into`
      auto prefetch_next = [&](int t0, int into) {
        int nt0 = t0 + TB, ns0 = s0, nBs = Bs;
        if (nt0 >= Bs) { ns0 = s0 + B; nt0 = 0; nBs = (n_tr - ns0) < B ? (n_tr - ns0) : B; }
        if (ns0 < n_tr) {
          const int nnb = (nBs - nt0) < TB ? (nBs - nt0) : TB;
          const uint16_t* rows = v.order + ns0 + nt0;
          stage_rows_async(a, a.X, a.y, v, dp, into, nnb, [&](int r) { return (int)rows[r]; }, tid, nt);
        }
      };

      if constexpr (!PL) {
        for (int t0 = 0; t0 < Bs; t0 += TB) {
          const int nb = (Bs - t0) < TB ? (Bs - t0) : TB;
          // rows of this sub-tile have landed; everyone is past the previous gW1 phase
          cp_async_wait_all();
          __syncthreads();
          BBO_PHASE(2);
          const float* xs = v.Xs + buf * TB * dp;
          const float* ysb = v.ys + buf * TB;
          prefetch_next(t0, buf ^ 1);
          forward_hidden<LEAN>(v, L, xs, d, dp, Hs, nb, tid, nt);
          __syncthreads();
          BBO_PHASE(3);
          output_phase(v.A1, ysb, nb, t0, 0, n_warps);
          __syncthreads();
          BBO_PHASE(4);
          unit_phase(v.A1, nb);
          __syncthreads();
          BBO_PHASE(5);
          gw1_phase(xs, v.A1, nb);
          buf ^= 1;
          BBO_PHASE(6);
        }
      } else {
        // Pipelined schedule: the gradient tiles of sub-tile t-1 are accumulated while the extra
        // warps (which own no tile and no hidden unit) run the output layer of sub-tile t.  Three
        // row buffers (t-1 for the gradient, t for the forward pass, t+1 in flight) and two
        // activation buffers make the two independent.  Every accumulator still receives its
        // rows in ascending order: each is owned by one thread, which visits the sub-tiles in order.
        const int T = (Bs + TB - 1) / TB;
        for (int i = 0; i <= T; ++i) {
          const int t0 = i * TB;
          const int nb = i < T ? ((Bs - t0) < TB ? (Bs - t0) : TB) : 0;
          cp_async_wait_all();
          __syncthreads();  // rows of sub-tile i have landed; everyone is past the unit phase of i-1
          BBO_PHASE(2);
          const int xb = buf, xb_prev = buf == 0 ? 2 : buf - 1, xb_next = buf == 2 ? 0 : buf + 1;
          float* A1cur = v.A1 + abuf * TB * L.WP;
          float* A1prev = v.A1 + (abuf ^ 1) * TB * L.WP;
          const float* ysb = v.ys + xb * TB;
          if (i < T) {
            prefetch_next(t0, xb_next);
            if (tid < nt_main) {
              FitView vv = v;
              vv.A1 = A1cur;
              forward_hidden<LEAN>(vv, L, v.Xs + xb * TB * dp, d, dp, Hs, nb, tid, nt_main);
            }
          }
          __syncthreads();
          BBO_PHASE(3);
          if (i < T && warp >= out_w0) output_phase(A1cur, ysb, nb, t0, out_w0, n_warps - out_w0);
          if (i > 0) {
            const int pnb = (Bs - (t0 - TB)) < TB ? (Bs - (t0 - TB)) : TB;
            gw1_phase(v.Xs + xb_prev * TB * dp, A1prev, pnb);
          }
          __syncthreads();
          BBO_PHASE(6);
          if (i < T) {
            unit_phase(A1cur, nb);
            buf = xb_next;
            abuf ^= 1;
          }
          BBO_PHASE(5);
        }
      }
      __syncthreads();  // A1 / D2 / W reads of this step are done; step size is visible
      BBO_PHASE(7);

      // ---- loss trace (debug): row losses in ascending order plus the L2 term ----
      if (want_loss) {
        float sq = 0.f;
        for (int k = 0; k < d; ++k)
          for (int j = tid; j < H; j += nt) { const float w = v.W[L.oW1 + k * Hs + j]; sq = __fmaf_rn(w, w, sq); }
        for (int j = tid; j < H; j += nt)
          for (int o = 0; o < CT; ++o) { const float w = v.W[L.oW2 + o * L.WP + j]; sq = __fmaf_rn(w, w, sq); }
        for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        if (lane == 0) sh.red[warp] = sq;
        __syncthreads();
        if (tid == 0) {
          float tot = 0.f;
          for (int w = 0; w < n_warps; ++w) tot += sh.red[w];
          float ls = 0.f;
          for (int b = 0; b < Bs; ++b) ls = __fadd_rn(ls, v.lossb[b]);
          const float loss = __fadd_rn(__fmul_rn(ls, invB), __fmul_rn(__fmul_rn(__fmul_rn(0.5f, c.alpha), invB), tot));
          a.trace[((size_t)config * a.K + fold) * a.trace_steps + step_no] = loss;
        }
      }

      // ---- L2 term and Adam, by the owner of each gradient ----
      const float step = sh.step[step_no & 1];
      const bool sgd = a.solver == 1;
      if (tile_warp) {
        // Every lane of a tile-owner warp walks the eight tile rows, two at a time (the
        // tensor-memory accesses are warp-wide); lanes without a tile, and rows k >= d, touch only
        // their own moments.  Two rows give sixteen independent update chains, which is what
        // keeps a lone warp's pipeline busy.  (Requesting the next pair's moments ahead of the
        // update cost 32 registers and gained nothing.)  The gradient tile is consumed: it is
        // zeroed at the start of the next step anyway.
        uint32_t mr[16], vr[16];
        auto next_rows = [&]() {  // rows 2, 3, .. of the gradient tile move up by two
#pragma unroll
          for (int r = 0; r < 6; ++r)
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) g1[r][cc] = g1[r + 2][cc];
        };
        auto pair_update = [&](int pr, auto R0) {  // rows 2 pr, 2 pr + 1 of the tile, held in g1[r0], g1[r0 + 1]
          constexpr int r0 = decltype(R0)::value;
          const int i0 = 2 * pr;
          const bool live0 = has_tile && (k0 + i0) < d, live1 = has_tile && (k0 + i0 + 1) < d;
          if constexpr (DPC == 0) {
            // Feature counts that are not a multiple of eight leave padding rows in the last row
            // block; where a row pair is padding for every lane of the warp (always so when d < 8)
            // its moments stay zero and the pair is skipped.
            if (__all_sync(0xffffffffu, !live0 && !live1)) return;
          }
          const int offA = L.oW1 + (k0 + i0) * Hs + jA, offB = L.oW1 + (k0 + i0) * Hs + jB;
          float w16[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) w16[j] = 0.f;
          auto load_w = [&]() {
            if (live0) {
              const float4 wA = *reinterpret_cast<float4*>(v.W + offA), wB = *reinterpret_cast<float4*>(v.W + offB);
              w16[0] = wA.x; w16[1] = wA.y; w16[2] = wA.z; w16[3] = wA.w; w16[4] = wB.x; w16[5] = wB.y; w16[6] = wB.z; w16[7] = wB.w;
            }
            if (live1) {
              const float4 wA = *reinterpret_cast<float4*>(v.W + offA + Hs), wB = *reinterpret_cast<float4*>(v.W + offB + Hs);
              w16[8] = wA.x; w16[9] = wA.y; w16[10] = wA.z; w16[11] = wA.w; w16[12] = wB.x; w16[13] = wB.y; w16[14] = wB.z; w16[15] = wB.w;
            }
          };
          tmem_load16_issue(tm + 16u * pr, mr);
          tmem_load16_issue(tm + 64u + 16u * pr, vr);
          load_w();
          tmem_wait_loads16(mr, vr);
          float m16[16], v16[16], g16[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            m16[j] = __uint_as_float(mr[j]); v16[j] = __uint_as_float(vr[j]);
            g16[j] = __fmaf_rn(aB, w16[j], g1[r0 + (j >> 3)][j & 7]);
          }
          if (sgd) {
            sgd_group<16>(w16, m16, g16, c.lr, beta1);
          } else if (!adam_group_fast<16>(w16, m16, v16, g16, beta1, beta2, omb1, omb2, step, eps, eps_safe)) {
            // not certified: redo the parameter update from the stored weights with the IEEE routines
            load_w();
            adam_params_ieee<16>(w16, m16, v16, step, eps);
          }
          if (live0) {
            *reinterpret_cast<float4*>(v.W + offA) = make_float4(w16[0], w16[1], w16[2], w16[3]);
            *reinterpret_cast<float4*>(v.W + offB) = make_float4(w16[4], w16[5], w16[6], w16[7]);
          }
          if (live1) {
            *reinterpret_cast<float4*>(v.W + offA + Hs) = make_float4(w16[8], w16[9], w16[10], w16[11]);
            *reinterpret_cast<float4*>(v.W + offB + Hs) = make_float4(w16[12], w16[13], w16[14], w16[15]);
          }
          tmem_store16(tm + 16u * pr, m16);
          tmem_store16(tm + 64u + 16u * pr, v16);
        };
        // The pair loop is rolled, with the tile's rows moved up between iterations (register
        // arrays cannot be indexed by the loop counter): unrolled it is 35 KB of code that runs
        // once per step, and CTAs of different widths on one SM, running different instances,
        // were starving each other of instructions.  Register-capped instances roll two pairs
        // per iteration (one pair per iteration cost them 5 to 8 %).
        if constexpr (!LEAN) {
#pragma unroll 1
          for (int pr = 0; pr < 4; ++pr) {
            pair_update(pr, std::integral_constant<int, 0>{});
            next_rows();
          }
        } else {
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) {
            pair_update(2 * hf, std::integral_constant<int, 0>{});
            pair_update(2 * hf + 1, std::integral_constant<int, 2>{});
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
              for (int cc = 0; cc < 8; ++cc) g1[r][cc] = g1[r + 4][cc];
          }
        }
        tmem_wait_stores();
      }
      if (unit_role) {
        float wu[CT + 1], mu[CT + 1], vu[CT + 1], gu[CT + 1], wold[CT + 1];
#pragma unroll
        for (int o = 0; o < CT; ++o) {
          const int off = L.oW2 + o * L.WP + tid;
          wu[o] = w2[o]; mu[o] = v.M[off]; vu[o] = v.V[off];
          gu[o] = __fmaf_rn(aB, w2[o], g2[o]);
        }
        wu[CT] = v.W[L.ob1 + tid]; mu[CT] = v.M[L.ob1 + tid]; vu[CT] = v.V[L.ob1 + tid]; gu[CT] = gb1;
#pragma unroll
        for (int o = 0; o <= CT; ++o) wold[o] = wu[o];
        if (sgd) {
          sgd_group<CT + 1>(wu, mu, gu, c.lr, beta1);
        } else if (!adam_group_fast<CT + 1>(wu, mu, vu, gu, beta1, beta2, omb1, omb2, step, eps, eps_safe)) {
#pragma unroll
          for (int o = 0; o <= CT; ++o) wu[o] = wold[o];
          adam_params_ieee<CT + 1>(wu, mu, vu, step, eps);
        }
#pragma unroll
        for (int o = 0; o < CT; ++o) {
          const int off = L.oW2 + o * L.WP + tid;
          v.W[off] = wu[o]; v.M[off] = mu[o]; v.V[off] = vu[o];
        }
        v.W[L.ob1 + tid] = wu[CT]; v.M[L.ob1 + tid] = mu[CT]; v.V[L.ob1 + tid] = vu[CT];
      }
      if (o_role) {
        const int off = L.ob2 + oo;
        if (sgd) {
          float w1[1] = {v.W[off]}, m1[1] = {v.M[off]};
          const float g1b[1] = {gb2};
          sgd_group<1>(w1, m1, g1b, c.lr, beta1);
          v.W[off] = w1[0]; v.M[off] = m1[0];
        } else {
          float w1[1] = {v.W[off]}, m1[1] = {v.M[off]}, v1[1] = {v.V[off]};
          const float g1b[1] = {gb2};
          const float wold = w1[0];
          if (!adam_group_fast<1>(w1, m1, v1, g1b, beta1, beta2, omb1, omb2, step, eps, eps_safe)) {
            w1[0] = wold;
            adam_params_ieee<1>(w1, m1, v1, step, eps);
          }
          v.W[off] = w1[0]; v.M[off] = m1[0]; v.V[off] = v1[0];
        }
      }
      ++step_no;
      BBO_PHASE(8);
      // the barrier at the top of the next sub-tile (or after the epoch) orders these writes
    }
    __syncthreads();
  }

  BBO_PHASE(2);
  // ---- held-out score ----
  if (tid == 0) { sh.correct = 0; sh.sq = 0.f; }
  __syncthreads();
  for (int t0 = 0; t0 < vs; t0 += TB) {
    const int nb = (vs - t0) < TB ? (vs - t0) : TB;
    if (holdout) stage_rows_async(a, a.Xt, a.yt, v, dp, 0, nb, [&](int r) { return t0 + r; }, tid, nt);
    else stage_rows_async(a, a.X, a.y, v, dp, 0, nb, [&](int r) { return a.pi[vb + t0 + r]; }, tid, nt);
    cp_async_wait_all();
    __syncthreads();
    forward_hidden<LEAN>(v, L, v.Xs, d, dp, Hs, nb, tid, nt);
    __syncthreads();
    for (int r0 = warp * 16; r0 < nb; r0 += n_warps * 16) {  // warp-uniform
      const int brow = r0 + (lane >> 1);
      const bool act = brow < nb;
      float z[QA];
      output_logits<CT>(v, L, H, ol, act ? brow : nb - 1, z);
      if (a.task == 0 && a.metric == 1) {
        // negative log-likelihood of the true class, written by the lane that holds its logit
        float mx, sum, ex[QA];
        softmax_scan<CT>(ol, z, mx, ex, sum);
        const int label = act ? (int)v.ys[brow] : -1;
#pragma unroll
        for (int q = 0; q < QA; ++q)
          if (q < ol.nq && ol.o0 + q == label) v.D2[brow * CS] = __fsub_rn(logf(sum), __fsub_rn(z[q], mx));
      } else if (a.task == 0) {
        // prediction: ascending scan with strict >, started by the even lane, finished by the odd one
        float best = z[0];
        int besti = ol.o0;
#pragma unroll
        for (int q = 1; q < QA; ++q) if (!ol.half && z[q] > best) { best = z[q]; besti = q; }
        const float b_even = __shfl_sync(0xffffffffu, best, lane & ~1);
        const int i_even = __shfl_sync(0xffffffffu, besti, lane & ~1);
        if (ol.half) {
          best = b_even;
          besti = i_even;
#pragma unroll
          for (int q = 0; q < QA; ++q) if (q < ol.nq && z[q] > best) { best = z[q]; besti = ol.o0 + q; }
          if (act && besti == (int)v.ys[brow]) atomicAdd(&sh.correct, 1);
        }
      } else if (act && !ol.half) {
        v.D2[brow * CS] = __fsub_rn(z[0], v.ys[brow]);
      }
    }
    __syncthreads();
    if ((a.task != 0 || a.metric == 1) && tid == 0) {  // row sums in ascending row order
      float sq = sh.sq;
      if (a.metric == 1) for (int b = 0; b < nb; ++b) sq = __fadd_rn(sq, fabsf(v.D2[b * CS]));
      else for (int b = 0; b < nb; ++b) { const float r = v.D2[b * CS]; sq = __fmaf_rn(r, r, sq); }
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
    a.fold_scores[(size_t)config * a.K + fold] = score;
  }
  BBO_PHASE(9);
#ifdef BBO_PHASE_TIMERS
  if (tid == 0 && q == 0)
    printf("PH Hs=%d H=%d B=%d nt=%d steps=%d | init %lld sort %lld wait %lld hidden %lld output %lld unit %lld gw1 %lld endbar %lld adam %lld score %lld\n",
           Hs, H, B, nt, step_no, sh.phase[0], sh.phase[1], sh.phase[2], sh.phase[3], sh.phase[4], sh.phase[5], sh.phase[6],
           sh.phase[7], sh.phase[8], sh.phase[9]);
#endif
  if (a.keep_theta != nullptr && config == a.n_configs - 1 && fold == a.K - 1) {
    const int n1 = d * H, n2 = H * CT;
    for (int i = tid; i < n1; i += nt) a.keep_theta[i] = v.W[L.oW1 + (i / H) * Hs + (i % H)];
    for (int i = tid; i < H; i += nt) a.keep_theta[n1 + i] = v.W[L.ob1 + i];
    for (int i = tid; i < n2; i += nt) a.keep_theta[n1 + H + i] = v.W[L.oW2 + (i % CT) * L.WP + (i / CT)];
    for (int i = tid; i < CT; i += nt) a.keep_theta[n1 + H + n2 + i] = v.W[L.ob2 + i];
  }
  tmem_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(sh.tmem_base, (uint32_t)a.tmem_cols);
}

// One CTA per fit; blockIdx.x indexes this launch's fit list (costliest first).
// The launch bounds cap the registers at 65,536 / (MINB x NTMAX); a scheduler's quarter of the
// register file holds two warps at 255 registers, so instances built for more than eight
// resident warps get about 168 and take the lean forms of the tile loops.
template <int CT, int HSC, int DPC, int NTMAX, int MINB, bool PL = false>
__global__ void __launch_bounds__(NTMAX, MINB) mlp_cv_fit_kernel(const FitArgs a) {
  extern __shared__ __align__(16) float smem[];
  __shared__ BlockShared sh;
  run_fit<CT, HSC, DPC, PL, (MINB * NTMAX > 256)>(a, blockIdx.x, smem, sh);
}

}  // namespace bbo
