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
// Work decomposition per minibatch, in sub-tiles of TB rows (H padded to Hs = 8*ceil(H/8)):
//   stage   cp.async gather of the next sub-tile's rows, double buffered
//   hidden  4x4 register tiles of A1 = relu(X W1 + b1), k ascending
//   output  one lane per z2[b][o] (32/C rows per warp), j ascending, softmax and loss
//           derivative with warp shuffles in the same lanes
//   gW2     two threads per hidden unit, each half of the classes, b ascending, in registers
//   delta1  4x4 register tiles (columns strided by Hs/4), o ascending, in place over A1
//   gW1     4x8 register tiles that persist across sub-tiles, b ascending; the owner applies
//           the L2 term and Adam to exactly its elements (second moments of W1 may stay in
//           the owner's registers for the whole fit)
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "device_math.cuh"
#include "fit_common.cuh"

namespace bbo {

struct FitView {  // per-fit pointers into shared memory
  float *W, *M, *V;     // V is biased so that V[off] is valid for off >= ob1 when W1's v is in registers
  uint16_t* order;
  float *lossb, *ys, *D2, *Xs, *A1;
  uint64_t* keys;
};

// Asynchronous gather of nb dataset rows into buffer `buf` of Xs / ys.  Rows nb..TB-1 are
// zero-filled so that the forward tiles read defined values.  row_of(r) = dataset row.
template <typename RowFn>
__device__ __forceinline__ void stage_rows_async(const FitArgs& a, const FitView& v, int buf, int nb,
                                                 RowFn row_of, int tid, int nt) {
  const int vec = a.dp >> 2;
  float* xs = v.Xs + buf * a.TB * a.dp;
  for (int i = tid; i < a.TB * vec; i += nt) {
    const int r = i / vec, q = i - r * vec;
    float4* dst = reinterpret_cast<float4*>(xs) + i;
    if (r < nb) cp_async_16(dst, reinterpret_cast<const float4*>(a.X + (size_t)row_of(r) * a.dp) + q);
    else *dst = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int r = tid; r < nb; r += nt) cp_async_4(v.ys + buf * a.TB + r, a.y + row_of(r));
  cp_async_commit();
}

// A1 = relu(Xs W1 + b1) for the TB-row tile; each thread owns 4x4 outputs, k ascending.
__device__ __forceinline__ void forward_hidden(const FitArgs& a, const FitView& v, const Layout& L,
                                               const float* xs, int nb, int tid, int nt) {
  const int JG = L.Hs >> 2, n_tiles = ((nb + 3) >> 2) * JG;
  const float* W1 = v.W + L.oW1;
  const int d4 = a.d >> 2, dp = a.dp, Hs = L.Hs;
  for (int t = tid; t < n_tiles; t += nt) {
    const int bg = t / JG, jg = t - bg * JG;
    const int b0 = bg << 2, j0 = jg << 2;
    const float4 bias = *reinterpret_cast<const float4*>(v.W + L.ob1 + j0);
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { acc[i][0] = bias.x; acc[i][1] = bias.y; acc[i][2] = bias.z; acc[i][3] = bias.w; }
    const float* xrow = xs + b0 * dp;
    const float* wp = W1 + j0;
    for (int k4 = 0; k4 < d4; ++k4) {
      float4 xv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const float4*>(xrow + i * dp + 4 * k4);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 w = *reinterpret_cast<const float4*>(wp + (4 * k4 + kk) * Hs);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float x = kk == 0 ? xv[i].x : (kk == 1 ? xv[i].y : (kk == 2 ? xv[i].z : xv[i].w));
          acc[i][0] = __fmaf_rn(x, w.x, acc[i][0]);
          acc[i][1] = __fmaf_rn(x, w.y, acc[i][1]);
          acc[i][2] = __fmaf_rn(x, w.z, acc[i][2]);
          acc[i][3] = __fmaf_rn(x, w.w, acc[i][3]);
        }
      }
    }
    for (int k = d4 << 2; k < a.d; ++k) {
      const float4 w = *reinterpret_cast<const float4*>(wp + k * Hs);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float x = xrow[i * dp + k];
        acc[i][0] = __fmaf_rn(x, w.x, acc[i][0]);
        acc[i][1] = __fmaf_rn(x, w.y, acc[i][1]);
        acc[i][2] = __fmaf_rn(x, w.z, acc[i][2]);
        acc[i][3] = __fmaf_rn(x, w.w, acc[i][3]);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float4 o;
      o.x = acc[i][0] > 0.f ? acc[i][0] : 0.f;
      o.y = acc[i][1] > 0.f ? acc[i][1] : 0.f;
      o.z = acc[i][2] > 0.f ? acc[i][2] : 0.f;
      o.w = acc[i][3] > 0.f ? acc[i][3] : 0.f;
      *reinterpret_cast<float4*>(v.A1 + (b0 + i) * Hs + j0) = o;
    }
  }
}

// z2[b][o] = b2[o] + sum_j A1[b][j] W2[j][o], j ascending, for lane (r, o) of a warp that
// holds 32/CT rows.  Returns the lane's logit (undefined for inactive lanes).
template <int CT>
__device__ __forceinline__ float output_logit(const FitView& v, const Layout& L, int CS, int H, int b, int o,
                                              bool active) {
  if (!active) return 0.f;
  float acc = v.W[L.ob2 + o];
  const float* arow = v.A1 + b * L.Hs;
  const float* wcol = v.W + L.oW2 + o;
  int j = 0;
  for (; j + 8 <= H; j += 8) {
    float av[8], wv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { av[u] = arow[j + u]; wv[u] = wcol[(j + u) * CS]; }
#pragma unroll
    for (int u = 0; u < 8; ++u) acc = __fmaf_rn(av[u], wv[u], acc);
  }
  for (; j < H; ++j) acc = __fmaf_rn(arow[j], wcol[j * CS], acc);
  return acc;
}

// Adam on one parameter with its gradient (L2 term already added for weights).
__device__ __forceinline__ void adam_one(float& th, float& m, float& vv, float g, float beta1, float beta2,
                                         float omb1, float omb2, float step, float eps) {
  m = __fmaf_rn(beta1, m, __fmul_rn(omb1, g));
  vv = __fmaf_rn(beta2, vv, __fmul_rn(__fmul_rn(omb2, g), g));
  th = __fsub_rn(th, __fmul_rn(step, __fdiv_rn(m, __fadd_rn(__fsqrt_rn(vv), eps))));
}

struct BlockShared {  // block-wide scalars
  float step[2];  // Adam step size, indexed by step parity (writer runs ahead of readers)
  int correct;
  float sq;
  float red[32];
};

// The whole fit.  CT: class count (compile time).  VR: second moments of W1 in registers.
template <int CT, bool VR>
__device__ __forceinline__ void run_fit(const FitArgs& a, int q, float* smem, BlockShared& sh) {
  constexpr int RW = 32 / CT;           // rows per warp in the output phase
  constexpr int CA = (CT + 1) / 2;      // classes per thread in the gW2 phase
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, n_warps = nt >> 5;
  const int2 cf = a.fits[q];
  const int config = cf.x, fold = cf.y;
  const Config c = a.configs[config];
  const int H = c.hidden, d = a.d, dp = a.dp, CS = a.CS, TB = a.TB;
  const Layout L(d, a.Hs, CS);
  const int Hs = L.Hs;
  int vb, vs;
  fold_segment(a.n, a.K, fold, &vb, &vs);
  const int n_tr = a.n - vs;
  const int B = c.batch_size < n_tr ? c.batch_size : n_tr;

  FitView v;
  v.W = smem;
  v.M = v.W + L.PS;
  v.V = VR ? (v.M + L.PS - L.ob1) : (v.M + L.PS);
  char* p = reinterpret_cast<char*>(v.M + L.PS + (VR ? L.PT : L.PS));
  v.order = reinterpret_cast<uint16_t*>(p); p += a.order_bytes;
  v.lossb = reinterpret_cast<float*>(p);    p += round_up(4 * a.loss_cap, 16);
  v.ys = reinterpret_cast<float*>(p);       p += 8 * TB;
  v.D2 = reinterpret_cast<float*>(p);       p += 4 * TB * CS;
  v.Xs = reinterpret_cast<float*>(p);
  v.A1 = v.Xs + 2 * TB * dp;
  v.keys = reinterpret_cast<uint64_t*>(p);

  // ---- initialisation: Glorot-uniform parameters, zero moments ----
  {
    const int n_zero = 2 * L.PS + (VR ? L.PT : L.PS);
    for (int i = tid; i < n_zero; i += nt) v.W[i] = 0.f;
  }
  __syncthreads();
  {
    const float bound1 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(d + H)));
    const float bound2 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(H + CT)));
    const int n1 = d * H, n2 = H * CT;
    for (int blk = tid; blk < ((n1 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 0u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n1) { const int k = idx / H, j = idx - k * H; v.W[L.oW1 + k * Hs + j] = glorot_value(word_of(r, w), bound1); }
      }
    }
    for (int blk = tid; blk < ((H + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 1u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int j = 4 * blk + w; if (j < H) v.W[L.ob1 + j] = glorot_value(word_of(r, w), bound1); }
    }
    for (int blk = tid; blk < ((n2 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 2u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n2) { const int j = idx / CT, o = idx - j * CT; v.W[L.oW2 + j * CS + o] = glorot_value(word_of(r, w), bound2); }
      }
    }
    for (int blk = tid; blk < ((CT + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 3u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int o = 4 * blk + w; if (o < CT) v.W[L.ob2 + o] = glorot_value(word_of(r, w), bound2); }
    }
  }
  __syncthreads();

  // ---- thread roles ----
  const int KG = dp >> 2, JG8 = Hs >> 3, JG4 = Hs >> 2;
  const bool has_tile = tid < KG * JG8;            // gW1 tile owner (host guarantees KG*JG8 <= nt)
  const int kg = has_tile ? tid / JG8 : 0, jg = has_tile ? tid - kg * JG8 : 0;
  const int k0 = kg << 2, jA = jg << 2, jB = (jg + JG8) << 2;
  const bool bias_owner = has_tile && kg == 0;     // also owns gb1 of its eight columns
  const int hj = tid >> 1, part = tid & 1;          // gW2: hidden unit and class half
  const bool w2_role = hj < H && (CT > 1 || part == 0);
  const int oa = part * CA;                         // first class of this thread's half
  const bool o_role = tid < CT;                     // gb2 owner
  // output phase: lane (r, o)
  const int orow = lane / CT, ocol = lane - orow * CT, obase = orow < RW ? orow * CT : 0;

  const float beta1 = c.beta1, beta2 = c.beta2, eps = c.eps;
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  double p1 = 1.0, p2 = 1.0;  // running beta^t (thread 0 only)
  int step_no = 0;
  float v1[4][8];             // second moments of this thread's W1 tile (VR only)
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) v1[i][j] = 0.f;

  for (int e = 0; e < c.epochs; ++e) {
    build_epoch_order(v.keys, v.order, a.pi, n_tr, vb, vs, a.seed, config, fold, e, tid, nt);
    // first sub-tile of the epoch
    int buf = 0;
    {
      const int Bs0 = n_tr < B ? n_tr : B, nb0 = Bs0 < TB ? Bs0 : TB;
      const uint16_t* rows = v.order;
      stage_rows_async(a, v, 0, nb0, [&](int r) { return (int)rows[r]; }, tid, nt);
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
      float g1[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) g1[i][j] = 0.f;
      float g2[CA], gb1[8], gb2 = 0.f;
#pragma unroll
      for (int o = 0; o < CA; ++o) g2[o] = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) gb1[j] = 0.f;

      for (int t0 = 0; t0 < Bs; t0 += TB) {
        const int nb = (Bs - t0) < TB ? (Bs - t0) : TB;
        // rows of this sub-tile have landed; everyone is past the previous gW1 phase
        cp_async_wait_all();
        __syncthreads();
        const float* xs = v.Xs + buf * TB * dp;
        const float* ysb = v.ys + buf * TB;
        {  // prefetch the next sub-tile of this epoch into the other buffer
          int nt0 = t0 + TB, ns0 = s0, nBs = Bs;
          if (nt0 >= Bs) { ns0 = s0 + B; nt0 = 0; nBs = (n_tr - ns0) < B ? (n_tr - ns0) : B; }
          if (ns0 < n_tr) {
            const int nnb = (nBs - nt0) < TB ? (nBs - nt0) : TB;
            const uint16_t* rows = v.order + ns0 + nt0;
            stage_rows_async(a, v, buf ^ 1, nnb, [&](int r) { return (int)rows[r]; }, tid, nt);
          }
        }
        forward_hidden(a, v, L, xs, nb, tid, nt);
        __syncthreads();

        // ---- output layer, softmax / residual, loss derivative (lanes own logits) ----
        for (int bw = warp * RW; bw < nb; bw += n_warps * RW) {
          const int b = bw + orow;
          const bool active = orow < RW && b < nb;
          const float z = output_logit<CT>(v, L, CS, H, b, ocol, active);
          const float yv = active ? ysb[b] : 0.f;
          float delta;
          if (a.task == 0) {
            const int label = (int)yv;
            float mx = __shfl_sync(0xffffffffu, z, obase);
#pragma unroll
            for (int o = 1; o < CT; ++o) { const float t = __shfl_sync(0xffffffffu, z, obase + o); if (t > mx) mx = t; }
            const float ex = spec_expf(__fsub_rn(z, mx));
            float sum = 0.f;
#pragma unroll
            for (int o = 0; o < CT; ++o) sum = __fadd_rn(sum, __shfl_sync(0xffffffffu, ex, obase + o));
            const float pr = __fdiv_rn(ex, sum);
            delta = __fmul_rn(__fsub_rn(pr, ocol == label ? 1.0f : 0.0f), invB);
            if (want_loss) {
              const float zl = __shfl_sync(0xffffffffu, z, obase + (active ? label : 0));
              if (active && ocol == 0) v.lossb[t0 + b] = __fsub_rn(logf(sum), __fsub_rn(zl, mx));
            }
          } else {
            const float r = __fsub_rn(z, yv);
            delta = __fmul_rn(r, invB);
            if (want_loss && active) v.lossb[t0 + b] = __fmul_rn(__fmul_rn(0.5f, r), r);
          }
          if (active) v.D2[b * CS + ocol] = delta;
        }
        __syncthreads();

        // ---- gW2[j][oa..oa+CA) += A1[b][j] * delta2[b][o], gb2[o] += delta2[b][o]; b ascending ----
        if (w2_role) {
          const float* ap = v.A1 + hj;
          const float* dp2 = v.D2 + oa;
#pragma unroll 4
          for (int b = 0; b < nb; ++b) {
            const float a1 = ap[b * Hs];
#pragma unroll
            for (int o = 0; o < CA; ++o)
              if (oa + o < CT) g2[o] = __fmaf_rn(a1, dp2[b * CS + o], g2[o]);
          }
        }
        if (o_role) for (int b = 0; b < nb; ++b) gb2 = __fadd_rn(gb2, v.D2[b * CS + tid]);
        __syncthreads();

        // ---- delta1 = (delta2 W2^T) masked by A1 > 0, in place; 4 rows x 4 strided columns ----
        {
          const int n_tiles = ((nb + 3) >> 2) * JG4;
          for (int t = tid; t < n_tiles; t += nt) {
            const int bg = t / JG4, jl = t - bg * JG4, b0 = bg << 2;
            float acc[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) acc[i][jj] = 0.f;
#pragma unroll
            for (int o4 = 0; o4 < (CT + 3) / 4; ++o4) {
              float4 dl[4], w2[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) dl[i] = *reinterpret_cast<const float4*>(v.D2 + (b0 + i) * CS + 4 * o4);
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) w2[jj] = *reinterpret_cast<const float4*>(v.W + L.oW2 + (jl + jj * JG4) * CS + 4 * o4);
#pragma unroll
              for (int oo = 0; oo < 4; ++oo) {
                if (4 * o4 + oo < CT) {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const float dv = oo == 0 ? dl[i].x : (oo == 1 ? dl[i].y : (oo == 2 ? dl[i].z : dl[i].w));
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                      const float wv = oo == 0 ? w2[jj].x : (oo == 1 ? w2[jj].y : (oo == 2 ? w2[jj].z : w2[jj].w));
                      acc[i][jj] = __fmaf_rn(dv, wv, acc[i][jj]);
                    }
                  }
                }
              }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                float* cell = v.A1 + (b0 + i) * Hs + jl + jj * JG4;
                *cell = *cell > 0.f ? acc[i][jj] : 0.f;
              }
          }
        }
        __syncthreads();

        // ---- gW1 tile: rows k0..k0+3, columns jA..jA+3 and jB..jB+3, b ascending; gb1 ----
        if (has_tile) {
          const float* xp = xs + k0;
          const float* da = v.A1 + jA;
          const float* db = v.A1 + jB;
#pragma unroll 2
          for (int b = 0; b < nb; ++b) {
            const float4 xv = *reinterpret_cast<const float4*>(xp + b * dp);
            const float4 dA = *reinterpret_cast<const float4*>(da + b * Hs);
            const float4 dB = *reinterpret_cast<const float4*>(db + b * Hs);
            const float xk[4] = {xv.x, xv.y, xv.z, xv.w};
            const float ds[8] = {dA.x, dA.y, dA.z, dA.w, dB.x, dB.y, dB.z, dB.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 8; ++j) g1[i][j] = __fmaf_rn(xk[i], ds[j], g1[i][j]);
            if (bias_owner) {
#pragma unroll
              for (int j = 0; j < 8; ++j) gb1[j] = __fadd_rn(gb1[j], ds[j]);
            }
          }
        }
        buf ^= 1;
      }
      __syncthreads();  // A1 / D2 / W reads of this step are done; step size is visible

      // ---- loss trace (debug): row losses in ascending order plus the L2 term ----
      if (want_loss) {
        float sq = 0.f;
        for (int k = 0; k < d; ++k)
          for (int j = tid; j < H; j += nt) { const float w = v.W[L.oW1 + k * Hs + j]; sq = __fmaf_rn(w, w, sq); }
        for (int j = tid; j < H; j += nt)
          for (int o = 0; o < CT; ++o) { const float w = v.W[L.oW2 + j * CS + o]; sq = __fmaf_rn(w, w, sq); }
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
      if (has_tile) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int k = k0 + i;
          if (k < d) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int off = L.oW1 + k * Hs + (half ? jB : jA);
              float4 w = *reinterpret_cast<float4*>(v.W + off);
              float4 m = *reinterpret_cast<float4*>(v.M + off);
              float4 vv;
              if (VR) vv = make_float4(v1[i][4 * half], v1[i][4 * half + 1], v1[i][4 * half + 2], v1[i][4 * half + 3]);
              else vv = *reinterpret_cast<float4*>(v.V + off);
              const float* g = &g1[i][4 * half];
              adam_one(w.x, m.x, vv.x, __fmaf_rn(aB, w.x, g[0]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.y, m.y, vv.y, __fmaf_rn(aB, w.y, g[1]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.z, m.z, vv.z, __fmaf_rn(aB, w.z, g[2]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.w, m.w, vv.w, __fmaf_rn(aB, w.w, g[3]), beta1, beta2, omb1, omb2, step, eps);
              *reinterpret_cast<float4*>(v.W + off) = w;
              *reinterpret_cast<float4*>(v.M + off) = m;
              if (VR) { v1[i][4 * half] = vv.x; v1[i][4 * half + 1] = vv.y; v1[i][4 * half + 2] = vv.z; v1[i][4 * half + 3] = vv.w; }
              else *reinterpret_cast<float4*>(v.V + off) = vv;
            }
          }
        }
        if (bias_owner) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int col = (j < 4 ? jA : jB) + (j & 3);
            if (col < H) {
              const int off = L.ob1 + col;
              adam_one(v.W[off], v.M[off], v.V[off], gb1[j], beta1, beta2, omb1, omb2, step, eps);
            }
          }
        }
      }
      if (w2_role) {
#pragma unroll
        for (int o = 0; o < CA; ++o) {
          if (oa + o < CT) {
            const int off = L.oW2 + hj * CS + oa + o;
            float w = v.W[off];
            adam_one(w, v.M[off], v.V[off], __fmaf_rn(aB, w, g2[o]), beta1, beta2, omb1, omb2, step, eps);
            v.W[off] = w;
          }
        }
      }
      if (o_role) {
        const int off = L.ob2 + tid;
        adam_one(v.W[off], v.M[off], v.V[off], gb2, beta1, beta2, omb1, omb2, step, eps);
      }
      ++step_no;
      // the barrier at the top of the next sub-tile (or of the sort) orders these writes
    }
    __syncthreads();
  }

  // ---- held-out score ----
  if (tid == 0) { sh.correct = 0; sh.sq = 0.f; }
  __syncthreads();
  for (int t0 = 0; t0 < vs; t0 += TB) {
    const int nb = (vs - t0) < TB ? (vs - t0) : TB;
    stage_rows_async(a, v, 0, nb, [&](int r) { return a.pi[vb + t0 + r]; }, tid, nt);
    cp_async_wait_all();
    __syncthreads();
    forward_hidden(a, v, L, v.Xs, nb, tid, nt);
    __syncthreads();
    for (int bw = warp * RW; bw < nb; bw += n_warps * RW) {
      const int b = bw + orow;
      const bool active = orow < RW && b < nb;
      const float z = output_logit<CT>(v, L, CS, H, b, ocol, active);
      if (a.task == 0) {
        float best = __shfl_sync(0xffffffffu, z, obase);
        int besti = 0;
#pragma unroll
        for (int o = 1; o < CT; ++o) {
          const float t = __shfl_sync(0xffffffffu, z, obase + o);
          if (t > best) { best = t; besti = o; }
        }
        if (active && ocol == 0 && besti == (int)v.ys[b]) atomicAdd(&sh.correct, 1);
      } else if (active) {
        v.D2[b * CS] = __fsub_rn(z, v.ys[b]);
      }
    }
    __syncthreads();
    if (a.task != 0 && tid == 0) {
      float sq = sh.sq;
      for (int b = 0; b < nb; ++b) { const float r = v.D2[b * CS]; sq = __fmaf_rn(r, r, sq); }
      sh.sq = sq;
    }
    __syncthreads();
  }
  if (tid == 0) {
    float score;
    if (a.task == 0) {
      score = __fdiv_rn((float)sh.correct, (float)vs);
    } else {
      score = -__fdiv_rn(sh.sq, (float)vs);
      if (score != score) score = __int_as_float(0xFF800000);
    }
    a.fold_scores[(size_t)config * a.K + fold] = score;
  }
  if (a.keep_theta != nullptr && config == a.n_configs - 1 && fold == a.K - 1) {
    const int n1 = d * H, n2 = H * CT;
    for (int i = tid; i < n1; i += nt) a.keep_theta[i] = v.W[L.oW1 + (i / H) * Hs + (i % H)];
    for (int i = tid; i < H; i += nt) a.keep_theta[n1 + i] = v.W[L.ob1 + i];
    for (int i = tid; i < n2; i += nt) a.keep_theta[n1 + H + i] = v.W[L.oW2 + (i / CT) * CS + (i % CT)];
    for (int i = tid; i < CT; i += nt) a.keep_theta[n1 + H + n2 + i] = v.W[L.ob2 + i];
  }
}

// One CTA per fit; blockIdx.x indexes this launch's fit list (costliest first).
template <int CT, bool VR, int NTMAX, int MINB>
__global__ void __launch_bounds__(NTMAX, MINB) mlp_cv_fit_kernel(const FitArgs a) {
  extern __shared__ __align__(16) float smem[];
  __shared__ BlockShared sh;
  run_fit<CT, VR>(a, blockIdx.x, smem, sh);
}

}  // namespace bbo
