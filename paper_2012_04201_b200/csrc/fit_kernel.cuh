// One CTA trains and scores one (configuration, fold) fit with parameters and Adam moments
// resident in shared memory (paper sec. 2: the function evaluated is the cross-validation
// score of a model on a dataset; Table 1: MLP-adam, metrics acc / mse; sec. 5: the model
// evaluation is what runs on the GPU, with the data kept there).
//
// Arithmetic contract.  Every accumulation runs in one fixed order so that results do not
// depend on the thread mapping: forward sums ascend over the input index with fused
// multiply-adds starting from the bias; gradient sums ascend over the minibatch row starting
// from zero; the softmax uses the explicit exponential of device_math.cuh; division and
// square root are IEEE; the Adam bias-correction products are kept in binary64 and the step
// size is rounded to binary32 once per step.  Threads own outputs (never partial sums), so
// there is no split reduction anywhere on the training path.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "device_math.cuh"

namespace bbo {

struct Config {  // mirrors bbo_mlp_config (32 bytes)
  int32_t hidden, batch_size, epochs;
  float alpha, lr, beta1, beta2, eps;
};

struct FitArgs {
  const float* X;        // [n][dp], rows 16-byte aligned
  const float* y;        // [n]
  const int32_t* pi;     // [n] fold permutation
  const Config* configs; // [n_configs]
  const int2* fits;      // [n_fits] (configuration, fold), launch order
  float* fold_scores;    // [n_configs * K]
  float* trace;          // [n_configs * K * trace_steps] or null
  float* keep_theta;     // parameters of fit (n_configs-1, K-1) in dense layout, or null
  int32_t* queue;        // work counter
  int32_t n_fits, n_configs;
  int32_t n, d, dp, C, CS, K, task;
  int32_t TB;            // rows per sub-tile (multiple of 4)
  int32_t trace_steps, loss_cap;  // loss_cap: rows of the per-row loss buffer
  int32_t order_bytes;   // bytes reserved for the epoch order (uint16 per training row)
  uint64_t seed;
};

__host__ __device__ inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// Shared-memory layout of one fit (float offsets inside the parameter block).
struct Layout {
  int Hs, oW1, ob1, oW2, ob2, PS;
  __host__ __device__ Layout(int d, int H, int CS) {
    Hs = round_up(H, 8);
    oW1 = 0;
    ob1 = d * Hs;
    oW2 = ob1 + Hs;
    ob2 = oW2 + H * CS;
    PS = round_up(ob2 + CS, 4);
  }
};

__host__ __device__ inline int next_pow2(int x) {
  int p = 4;
  while (p < x) p <<= 1;
  return p;
}

// Bytes of scratch after the three parameter-sized blocks.
__host__ __device__ inline size_t scratch_bytes(int Hs, int dp, int CS, int TB, int order_bytes,
                                                int loss_cap, int n_sort) {
  size_t fixed = (size_t)order_bytes + (size_t)round_up(4 * loss_cap, 16) + 4u * TB + 4u * TB * CS;
  size_t xa = 4u * (size_t)TB * dp + 4u * (size_t)TB * Hs;
  size_t keys = 8u * (size_t)next_pow2(n_sort);
  return fixed + (xa > keys ? xa : keys);
}

__host__ __device__ inline void fold_segment(int n, int K, int f, int* begin, int* size) {
  const int base = n / K, rem = n % K;
  *begin = f * base + (f < rem ? f : rem);
  *size = base + (f < rem ? 1 : 0);
}

// Ascending bitonic sort of np2 (power of two) 64-bit keys in shared memory.
__device__ inline void bitonic_sort(uint64_t* keys, int np2, int tid, int nt) {
  for (int k = 2; k <= np2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = tid; t < (np2 >> 1); t += nt) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int l = i | j;
        const bool up = (i & k) == 0;
        const uint64_t a = keys[i], b = keys[l];
        if ((a > b) == up) { keys[i] = b; keys[l] = a; }
      }
      __syncthreads();
    }
  }
}

// Permutation of 0..N-1 by ascending (random word << 32 | index); result left in the low
// words of keys[0..N).  Leaves the block synchronised.
__device__ inline void sorted_keys(uint64_t* keys, int N, uint64_t seed, uint32_t stream, uint32_t a,
                                   uint32_t b, uint32_t c, int tid, int nt) {
  const int np2 = next_pow2(N);
  for (int blk = tid; blk < (np2 >> 2); blk += nt) {
    const uint4 r = philox4x32_10(seed, stream, a, b, c, (uint32_t)blk);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int i = 4 * blk + w;
      keys[i] = i < N ? ((uint64_t)word_of(r, w) << 32) | (uint32_t)i : ~0ull;
    }
  }
  __syncthreads();
  bitonic_sort(keys, np2, tid, nt);
}

// Dataset row visited i-th in epoch `epoch`: the epoch permutation applied to the training
// list (fold permutation with the held-out segment removed, order kept).
__device__ inline void build_epoch_order(uint64_t* keys, uint16_t* order, const int32_t* pi, int n_tr,
                                         int vb, int vs, uint64_t seed, uint32_t config, uint32_t fold,
                                         uint32_t epoch, int tid, int nt) {
  sorted_keys(keys, n_tr, seed, kStreamPerm, config, fold, epoch, tid, nt);
  for (int i = tid; i < n_tr; i += nt) {
    const int s = (int)(uint32_t)keys[i];
    order[i] = (uint16_t)pi[s < vb ? s : s + vs];
  }
  __syncthreads();
}

struct FitView {  // per-fit pointers into shared memory
  float *W, *M, *V;
  uint16_t* order;
  float *lossb, *ys, *D2, *Xs, *A1;
  uint64_t* keys;
};

// Stage nb dataset rows (ids from `rows`, or pi positions when scoring) into Xs / ys; rows
// nb..TB of the tile are zero-filled so that the forward tiles read defined values.
template <typename RowFn>
__device__ inline void stage_rows(const FitArgs& a, const FitView& v, int nb, RowFn row_of, int tid, int nt) {
  const int vec = a.dp >> 2;
  for (int i = tid; i < a.TB * vec; i += nt) {
    const int r = i / vec, q = i - r * vec;
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < nb) val = __ldg(reinterpret_cast<const float4*>(a.X + (size_t)row_of(r) * a.dp) + q);
    reinterpret_cast<float4*>(v.Xs)[i] = val;
  }
  for (int r = tid; r < nb; r += nt) v.ys[r] = __ldg(a.y + row_of(r));
}

// A1 = relu(Xs W1 + b1) for the TB-row tile; each thread owns 4x4 outputs, k ascending.
__device__ inline void forward_hidden(const FitArgs& a, const FitView& v, const Layout& L, int tid, int nt) {
  const int JG = L.Hs >> 2, n_tiles = (a.TB >> 2) * JG;
  const float* W1 = v.W + L.oW1;
  const int d4 = a.d >> 2;
  for (int t = tid; t < n_tiles; t += nt) {
    const int bg = t / JG, jg = t - bg * JG;
    const int b0 = bg << 2, j0 = jg << 2;
    const float4 bias = *reinterpret_cast<const float4*>(v.W + L.ob1 + j0);
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { acc[i][0] = bias.x; acc[i][1] = bias.y; acc[i][2] = bias.z; acc[i][3] = bias.w; }
    const float* xrow = v.Xs + b0 * a.dp;
    for (int k4 = 0; k4 < d4; ++k4) {
      float4 xv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const float4*>(xrow + i * a.dp + 4 * k4);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 w = *reinterpret_cast<const float4*>(W1 + (4 * k4 + kk) * L.Hs + j0);
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
      const float4 w = *reinterpret_cast<const float4*>(W1 + k * L.Hs + j0);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float x = xrow[i * a.dp + k];
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
      *reinterpret_cast<float4*>(v.A1 + (b0 + i) * L.Hs + j0) = o;
    }
  }
}

// Z2[b][o] = b2[o] + sum_j A1[b][j] W2[j][o], j ascending; one thread per output.
__device__ inline void forward_output(const FitArgs& a, const FitView& v, const Layout& L, int H, int nb,
                                      int tid, int nt) {
  const float* W2 = v.W + L.oW2;
  for (int idx = tid; idx < nb * a.C; idx += nt) {
    const int b = idx / a.C, o = idx - b * a.C;
    float acc = v.W[L.ob2 + o];
    const float* arow = v.A1 + b * L.Hs;
    const float* wcol = W2 + o;
#pragma unroll 4
    for (int j = 0; j < H; ++j) acc = __fmaf_rn(arow[j], wcol[j * a.CS], acc);
    v.D2[b * a.CS + o] = acc;
  }
}

// Row-wise loss derivative, in place over Z2: softmax minus one-hot, or the residual, times
// 1/Bs.  When want_loss, the row's loss goes to lossb[row_base + b].
__device__ inline void output_delta(const FitArgs& a, const FitView& v, int nb, float invB, bool want_loss,
                                    int row_base, int tid) {
  if (tid >= nb) return;
  float* z = v.D2 + tid * a.CS;
  const float yv = v.ys[tid];
  if (a.task == 0) {
    const int label = (int)yv;
    float mx = z[0];
    for (int o = 1; o < a.C; ++o) if (z[o] > mx) mx = z[o];
    const float zl = z[label];
    float sum = 0.f;
    for (int o = 0; o < a.C; ++o) {
      const float e = spec_expf(__fsub_rn(z[o], mx));
      z[o] = e;
      sum = __fadd_rn(sum, e);
    }
    for (int o = 0; o < a.C; ++o) {
      const float p = __fdiv_rn(z[o], sum);
      z[o] = __fmul_rn(__fsub_rn(p, o == label ? 1.0f : 0.0f), invB);
    }
    if (want_loss) v.lossb[row_base + tid] = __fsub_rn(logf(sum), __fsub_rn(zl, mx));
  } else {
    const float r = __fsub_rn(z[0], yv);
    z[0] = __fmul_rn(r, invB);
    if (want_loss) v.lossb[row_base + tid] = __fmul_rn(__fmul_rn(0.5f, r), r);
  }
}

// Adam on one parameter with its gradient (L2 term already added for weights).
__device__ __forceinline__ void adam_one(float& th, float& m, float& vv, float g, float beta1, float beta2,
                                         float omb1, float omb2, float step, float eps) {
  m = __fmaf_rn(beta1, m, __fmul_rn(omb1, g));
  vv = __fmaf_rn(beta2, vv, __fmul_rn(__fmul_rn(omb2, g), g));
  th = __fsub_rn(th, __fmul_rn(step, __fdiv_rn(m, __fadd_rn(__fsqrt_rn(vv), eps))));
}

struct StepShared {  // block-wide scalars
  float step;
  int correct;
  int fit;
  float red[32];
};

// The whole fit.  CT: compile-time bound on the class count (accumulators in registers).
template <int CT>
__device__ void run_fit(const FitArgs& a, int q, float* smem, StepShared& sh) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int2 cf = a.fits[q];
  const int config = cf.x, fold = cf.y;
  const Config c = a.configs[config];
  const int H = c.hidden, d = a.d, C = a.C, CS = a.CS, TB = a.TB;
  const Layout L(d, H, CS);
  int vb, vs;
  fold_segment(a.n, a.K, fold, &vb, &vs);
  const int n_tr = a.n - vs;
  const int B = c.batch_size < n_tr ? c.batch_size : n_tr;

  FitView v;
  v.W = smem;
  v.M = v.W + L.PS;
  v.V = v.M + L.PS;
  char* p = reinterpret_cast<char*>(v.V + L.PS);
  v.order = reinterpret_cast<uint16_t*>(p); p += a.order_bytes;
  v.lossb = reinterpret_cast<float*>(p);    p += round_up(4 * a.loss_cap, 16);
  v.ys = reinterpret_cast<float*>(p);       p += 4 * TB;
  v.D2 = reinterpret_cast<float*>(p);       p += 4 * TB * CS;
  v.Xs = reinterpret_cast<float*>(p);
  v.A1 = v.Xs + TB * a.dp;
  v.keys = reinterpret_cast<uint64_t*>(p);

  // ---- initialisation: Glorot-uniform parameters, zero moments ----
  for (int i = tid; i < 3 * L.PS; i += nt) v.W[i] = 0.f;
  __syncthreads();
  {
    const float bound1 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(d + H)));
    const float bound2 = __fsqrt_rn(__fdiv_rn(6.0f, (float)(H + C)));
    const int n1 = d * H, n2 = H * C;
    for (int blk = tid; blk < ((n1 + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 0u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int idx = 4 * blk + w;
        if (idx < n1) { const int k = idx / H, j = idx - k * H; v.W[L.oW1 + k * L.Hs + j] = glorot_value(word_of(r, w), bound1); }
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
        if (idx < n2) { const int j = idx / C, o = idx - j * C; v.W[L.oW2 + j * CS + o] = glorot_value(word_of(r, w), bound2); }
      }
    }
    for (int blk = tid; blk < ((C + 3) >> 2); blk += nt) {
      const uint4 r = philox4x32_10(a.seed, kStreamInit, config, fold, 3u, blk);
#pragma unroll
      for (int w = 0; w < 4; ++w) { const int o = 4 * blk + w; if (o < C) v.W[L.ob2 + o] = glorot_value(word_of(r, w), bound2); }
    }
  }
  __syncthreads();

  // ---- training ----
  const float beta1 = c.beta1, beta2 = c.beta2, eps = c.eps;
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  double p1 = 1.0, p2 = 1.0;  // running beta^t (thread 0 only)
  int step_no = 0;
  const int KG = a.dp >> 2, JG8 = L.Hs >> 3, n_gtiles = KG * JG8;
  const bool has_tile = tid < n_gtiles;
  const int kg = has_tile ? tid / JG8 : 0, jg = has_tile ? tid - kg * JG8 : 0;
  const int k0 = kg << 2, jA = jg << 2, jB = (jg + JG8) << 2;
  const bool j_role = tid < H;
  const bool o_role = tid < C;

  for (int e = 0; e < c.epochs; ++e) {
    build_epoch_order(v.keys, v.order, a.pi, n_tr, vb, vs, a.seed, config, fold, e, tid, nt);
    for (int s0 = 0; s0 < n_tr; s0 += B) {
      const int Bs = (n_tr - s0) < B ? (n_tr - s0) : B;
      const float invB = __fdiv_rn(1.0f, (float)Bs);
      const float aB = __fmul_rn(c.alpha, invB);
      const bool want_loss = a.trace != nullptr && step_no < a.trace_steps;
      if (tid == 0) {
        p1 *= (double)beta1;
        p2 *= (double)beta2;
        sh.step = (float)((double)c.lr * sqrt(1.0 - p2) / (1.0 - p1));
      }
      float g1[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) g1[i][j] = 0.f;
      float g2[CT], w2[CT];
      float gb1 = 0.f, gb2 = 0.f;
#pragma unroll
      for (int o = 0; o < CT; ++o) { g2[o] = 0.f; w2[o] = (j_role && o < C) ? v.W[L.oW2 + tid * CS + o] : 0.f; }

      for (int t0 = 0; t0 < Bs; t0 += TB) {
        const int nb = (Bs - t0) < TB ? (Bs - t0) : TB;
        const uint16_t* rows = v.order + s0 + t0;
        stage_rows(a, v, nb, [&](int r) { return (int)rows[r]; }, tid, nt);
        __syncthreads();
        forward_hidden(a, v, L, tid, nt);
        __syncthreads();
        forward_output(a, v, L, H, nb, tid, nt);
        __syncthreads();
        output_delta(a, v, nb, invB, want_loss, t0, tid);
        __syncthreads();
        // hidden unit j: gW2[j][:], delta1[:, j] (in place over A1), gb1[j]; output o: gb2[o]
        if (j_role) {
          for (int b = 0; b < nb; ++b) {
            const float a1 = v.A1[b * L.Hs + tid];
            const float* dl = v.D2 + b * CS;
            float acc = 0.f;
#pragma unroll
            for (int o = 0; o < CT; ++o) {
              if (o < C) {
                const float dv = dl[o];
                g2[o] = __fmaf_rn(a1, dv, g2[o]);
                acc = __fmaf_rn(dv, w2[o], acc);
              }
            }
            const float d1 = a1 > 0.f ? acc : 0.f;
            v.A1[b * L.Hs + tid] = d1;
            gb1 = __fadd_rn(gb1, d1);
          }
        } else if (tid < L.Hs) {
          for (int b = 0; b < nb; ++b) v.A1[b * L.Hs + tid] = 0.f;  // padded hidden columns
        }
        if (o_role) for (int b = 0; b < nb; ++b) gb2 = __fadd_rn(gb2, v.D2[b * CS + tid]);
        __syncthreads();
        // gW1 tile: rows k0..k0+3, columns jA..jA+3 and jB..jB+3, b ascending
        if (has_tile) {
          for (int b = 0; b < nb; ++b) {
            const float4 xv = *reinterpret_cast<const float4*>(v.Xs + b * a.dp + k0);
            const float4 dA = *reinterpret_cast<const float4*>(v.A1 + b * L.Hs + jA);
            const float4 dB = *reinterpret_cast<const float4*>(v.A1 + b * L.Hs + jB);
            const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
            const float ds[8] = {dA.x, dA.y, dA.z, dA.w, dB.x, dB.y, dB.z, dB.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 8; ++j) g1[i][j] = __fmaf_rn(xs[i], ds[j], g1[i][j]);
          }
        }
        __syncthreads();
      }

      // ---- loss trace (debug): row losses in ascending order plus the L2 term ----
      if (want_loss) {
        float sq = 0.f;
        for (int k = 0; k < d; ++k)
          for (int j = tid; j < H; j += nt) { const float w = v.W[L.oW1 + k * L.Hs + j]; sq = __fmaf_rn(w, w, sq); }
        for (int j = tid; j < H; j += nt)
          for (int o = 0; o < C; ++o) { const float w = v.W[L.oW2 + j * CS + o]; sq = __fmaf_rn(w, w, sq); }
        for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        if ((tid & 31) == 0) sh.red[tid >> 5] = sq;
        __syncthreads();
        if (tid == 0) {
          float tot = 0.f;
          for (int w = 0; w < ((nt + 31) >> 5); ++w) tot += sh.red[w];
          float ls = 0.f;
          for (int b = 0; b < Bs; ++b) ls = __fadd_rn(ls, v.lossb[b]);
          const float loss = __fadd_rn(__fmul_rn(ls, invB), __fmul_rn(__fmul_rn(__fmul_rn(0.5f, c.alpha), invB), tot));
          a.trace[((size_t)config * a.K + fold) * a.trace_steps + step_no] = loss;
        }
      }

      // ---- L2 term and Adam, by the owner of each gradient ----
      const float step = sh.step;  // written before the first barrier of this step
      if (has_tile) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int k = k0 + i;
          if (k < d) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int off = L.oW1 + k * L.Hs + (half ? jB : jA);
              float4 w = *reinterpret_cast<float4*>(v.W + off);
              float4 m = *reinterpret_cast<float4*>(v.M + off);
              float4 vv = *reinterpret_cast<float4*>(v.V + off);
              const float* g = &g1[i][4 * half];
              adam_one(w.x, m.x, vv.x, __fmaf_rn(aB, w.x, g[0]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.y, m.y, vv.y, __fmaf_rn(aB, w.y, g[1]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.z, m.z, vv.z, __fmaf_rn(aB, w.z, g[2]), beta1, beta2, omb1, omb2, step, eps);
              adam_one(w.w, m.w, vv.w, __fmaf_rn(aB, w.w, g[3]), beta1, beta2, omb1, omb2, step, eps);
              *reinterpret_cast<float4*>(v.W + off) = w;
              *reinterpret_cast<float4*>(v.M + off) = m;
              *reinterpret_cast<float4*>(v.V + off) = vv;
            }
          }
        }
      }
      if (j_role) {
#pragma unroll
        for (int o = 0; o < CT; ++o) {
          if (o < C) {
            const int off = L.oW2 + tid * CS + o;
            float w = w2[o];
            adam_one(w, v.M[off], v.V[off], __fmaf_rn(aB, w, g2[o]), beta1, beta2, omb1, omb2, step, eps);
            v.W[off] = w;
          }
        }
        const int off = L.ob1 + tid;
        adam_one(v.W[off], v.M[off], v.V[off], gb1, beta1, beta2, omb1, omb2, step, eps);
      }
      if (o_role) {
        const int off = L.ob2 + tid;
        adam_one(v.W[off], v.M[off], v.V[off], gb2, beta1, beta2, omb1, omb2, step, eps);
      }
      ++step_no;
      __syncthreads();
    }
  }

  // ---- held-out score ----
  if (tid == 0) sh.correct = 0;
  float sq = 0.f;  // thread 0: squared residuals in ascending row order
  __syncthreads();
  for (int t0 = 0; t0 < vs; t0 += TB) {
    const int nb = (vs - t0) < TB ? (vs - t0) : TB;
    stage_rows(a, v, nb, [&](int r) { return a.pi[vb + t0 + r]; }, tid, nt);
    __syncthreads();
    forward_hidden(a, v, L, tid, nt);
    __syncthreads();
    forward_output(a, v, L, H, nb, tid, nt);
    __syncthreads();
    if (a.task == 0) {
      if (tid < nb) {
        const float* z = v.D2 + tid * CS;
        int best = 0;
        for (int o = 1; o < C; ++o) if (z[o] > z[best]) best = o;
        if (best == (int)v.ys[tid]) atomicAdd(&sh.correct, 1);
      }
    } else if (tid == 0) {
      for (int b = 0; b < nb; ++b) {
        const float r = __fsub_rn(v.D2[b * CS], v.ys[b]);
        sq = __fmaf_rn(r, r, sq);
      }
    }
    __syncthreads();
  }
  if (tid == 0) {
    float score;
    if (a.task == 0) {
      score = __fdiv_rn((float)sh.correct, (float)vs);
    } else {
      score = -__fdiv_rn(sq, (float)vs);
      if (score != score) score = __int_as_float(0xFF800000);
    }
    a.fold_scores[(size_t)config * a.K + fold] = score;
  }
  if (a.keep_theta != nullptr && config == a.n_configs - 1 && fold == a.K - 1) {
    const int n1 = d * H, n2 = H * C;
    for (int i = tid; i < n1; i += nt) a.keep_theta[i] = v.W[L.oW1 + (i / H) * L.Hs + (i % H)];
    for (int i = tid; i < H; i += nt) a.keep_theta[n1 + i] = v.W[L.ob1 + i];
    for (int i = tid; i < n2; i += nt) a.keep_theta[n1 + H + i] = v.W[L.oW2 + (i / C) * CS + (i % C)];
    for (int i = tid; i < C; i += nt) a.keep_theta[n1 + H + n2 + i] = v.W[L.ob2 + i];
  }
  __syncthreads();
}

// Persistent CTAs pull fits from a counter in launch order (costliest first).
template <int CT, int NTB>
__global__ void __launch_bounds__(NTB, 1) mlp_cv_fit_kernel(const FitArgs a) {
  extern __shared__ __align__(16) float smem[];
  __shared__ StepShared sh;
  for (;;) {
    if (threadIdx.x == 0) sh.fit = atomicAdd(a.queue, 1);
    __syncthreads();
    const int q = sh.fit;
    __syncthreads();
    if (q >= a.n_fits) break;
    run_fit<CT>(a, q, smem, sh);
  }
}

// Fold split: pi = permutation of the rows by ascending (random word << 32 | row).
__global__ void fold_permutation_kernel(int n, uint64_t seed, int32_t* pi) {
  extern __shared__ __align__(16) float smem[];
  uint64_t* keys = reinterpret_cast<uint64_t*>(smem);
  sorted_keys(keys, n, seed, kStreamFold, 0u, 0u, 0u, threadIdx.x, blockDim.x);
  for (int i = threadIdx.x; i < n; i += blockDim.x) pi[i] = (int32_t)(uint32_t)keys[i];
}

// out[c] = (score[c][0] + ... + score[c][K-1]) / K, ascending fold.
__global__ void fold_mean_kernel(const float* fold_scores, int n_configs, int K, float* out) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_configs) return;
  float s = 0.f;
  for (int f = 0; f < K; ++f) s = __fadd_rn(s, fold_scores[(size_t)c * K + f]);
  out[c] = __fdiv_rn(s, (float)K);
}

// info[0] = max label, info[1] = 1 if any label is negative, fractional, huge or NaN.
__global__ void label_scan_kernel(const float* y, int n, int32_t* info) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const float v = y[i];
    if (!(v >= 0.f) || v != floorf(v) || v > 1.0e6f) atomicOr(&info[1], 1);
    else atomicMax(&info[0], (int)v);
  }
}

// Copy X into rows of dp floats (zero padded) so that every row starts 16-byte aligned.
__global__ void pad_rows_kernel(const float* X, int n, int d, int dp, float* out) {
  const size_t total = (size_t)n * dp;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / dp), k = (int)(i - (size_t)r * dp);
    out[i] = k < d ? X[(size_t)r * d + k] : 0.f;
  }
}

// Debug: epoch order of one fit written to global memory, and the fold of every row.
__global__ void debug_order_kernel(int n, int K, uint64_t seed, const int32_t* pi, int config, int fold,
                                   int epoch, int32_t* fold_of_row, int32_t* order_out) {
  extern __shared__ __align__(16) float smem[];
  int vb, vs;
  fold_segment(n, K, fold, &vb, &vs);
  const int n_tr = n - vs;
  uint16_t* order = reinterpret_cast<uint16_t*>(smem);
  uint64_t* keys = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(smem) + round_up(2 * n_tr, 16));
  build_epoch_order(keys, order, pi, n_tr, vb, vs, seed, config, fold, epoch, threadIdx.x, blockDim.x);
  for (int i = threadIdx.x; i < n_tr; i += blockDim.x) order_out[i] = order[i];
  for (int f = 0; f < K; ++f) {
    int b, s;
    fold_segment(n, K, f, &b, &s);
    for (int i = threadIdx.x; i < s; i += blockDim.x) fold_of_row[pi[b + i]] = f;
  }
}

__global__ void debug_rng_kernel(uint64_t seed, const uint32_t* ctr, int64_t count, uint32_t* out) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    const uint4 r = philox4x32_10(seed, ctr[5 * i], ctr[5 * i + 1], ctr[5 * i + 2], ctr[5 * i + 3], ctr[5 * i + 4]);
    out[4 * i] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
  }
}

__global__ void debug_exp_kernel(const float* x, int64_t count, float* out) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = spec_expf(x[i]);
}

}  // namespace bbo
