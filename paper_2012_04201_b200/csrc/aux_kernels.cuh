// Small kernels around the fit kernel: fold permutation, fold mean, label scan, row padding
// and the debug exports.  Included by exactly one translation unit.
#pragma once
#include "fit_common.cuh"

namespace bbo {

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
  __shared__ uint32_t red[32];
  uint16_t* order = reinterpret_cast<uint16_t*>(smem);
  void* scratch = reinterpret_cast<char*>(smem) + round_up(2 * n_tr, 16);
  build_epoch_order(scratch, red, order, pi, n_tr, vb, vs, seed, config, fold, epoch, threadIdx.x, blockDim.x);
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

// Debug: counts inputs in the safe range for which the branch-free square root / division
// differ from the IEEE intrinsics.  mode 0: sqrt(v) and sqrt(v) + eps over the bit patterns first .. first+count-1 (denormals included);
// mode 1: m / (sqrt(v) + eps) over `count` operand triples drawn from Philox words with
// exponents spread over the whole float range; mode 3: the same quotient with tiny or denormal
// m over ordinary v and eps, so that most quotients are denormal, exact ties included (a
// denominator of exactly 2 under an odd multiple of the smallest denormal).  out[0] = mismatches, out[1] = cases the fast
// path declared safe, out[2..3] = operands of one mismatch.
__global__ void debug_fast_math_kernel(int mode, uint64_t seed, uint64_t first, uint64_t count, unsigned long long* out) {
  unsigned long long bad = 0, safe_n = 0;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < count; i += (uint64_t)gridDim.x * blockDim.x) {
    if (mode == 0) {
      const float x = __uint_as_float((uint32_t)(first + i));
      if (!(x < 0x1p+32f)) continue;
      ++safe_n;
      const float eps = 0x1p-30f;
      const float a = adam_denominator_fast(x, eps), b = __fadd_rn(__fsqrt_rn(x), eps);
      const float a2 = __fmul_rn(sqrt_fast_rn(fmaxf(__fmul_rn(x, 0x1p+96f), 0x1p-60f)), 0x1p-48f), b2 = __fsqrt_rn(x);
      if (__float_as_uint(a) != __float_as_uint(b) || (x != 0.f && __float_as_uint(a2) != __float_as_uint(b2))) { ++bad; out[2] = __float_as_uint(x); }
    } else if (mode == 2) {  // softmax quotient: e = exp of a non-positive number, s in [1, 16]
      const uint4 r = philox4x32_10(seed, 8u, (uint32_t)(i >> 32), 0u, 0u, (uint32_t)i);
      const float e = spec_expf(-90.0f * (__uint2float_rn(r.x >> 8) * 0x1p-24f));
      const float s = __fadd_rn(1.0f, __fmul_rn(15.0f, __uint2float_rn(r.y >> 8) * 0x1p-24f));
      uint32_t safe = 1u;
      const float q = softmax_ratio_fast(e, s, safe);
      if (safe == 0u) continue;
      ++safe_n;
      const float ref = __fdiv_rn(e, s);
      if (__float_as_uint(q) != __float_as_uint(ref)) { ++bad; out[2] = __float_as_uint(e); out[3] = __float_as_uint(s); }
    } else if (mode == 3) {
      const uint4 r = philox4x32_10(seed, 9u, (uint32_t)(i >> 32), 0u, 0u, (uint32_t)i);
      float m = __uint_as_float((r.x & 0x807FFFFFu) | ((r.w % 48u) << 23));  // denormal .. 2^-80, either sign
      float vv = __uint_as_float((r.y & 0x007FFFFFu) | ((40u + (r.w >> 8) % 90u) << 23));  // 2^-87 .. 2^2
      if (((r.w >> 20) & 15u) == 0u) vv = __uint_as_float(r.y & 0x007FFFFFu);              // denormal or zero v
      const float eps_set[4] = {1e-8f, 0x1p-40f, 1e-3f, 0.75f};
      float eps = eps_set[(r.w >> 24) & 3u];
      if ((r.w >> 28) == 0u) {  // denominator exactly 2: odd numerators are exact ties
        vv = 1.5625f; eps = 0.75f;
        m = __uint_as_float((r.x & 0x80000000u) | (r.x & 0xFFu));
      }
      AdamCert cert;
      const float q = adam_ratio_fast(m, vv, eps, cert);
      if ((adam_eps_safe(eps) & cert.ok()) == 0u) continue;
      ++safe_n;
      const float ref = adam_ratio_ieee(m, vv, eps);
      if (__float_as_uint(q) != __float_as_uint(ref)) { ++bad; out[2] = __float_as_uint(m); out[3] = __float_as_uint(vv); }
    } else {
      const uint4 r = philox4x32_10(seed, 7u, (uint32_t)(i >> 32), 0u, 0u, (uint32_t)i);
      const float m = __uint_as_float(r.x);
      const float vv = __uint_as_float(r.y & 0x7FFFFFFFu);
      const float eps = __uint_as_float((r.z & 0x007FFFFFu) | ((20u + (r.w % 170u)) << 23));  // 2^-107 .. 2^62
      AdamCert cert;
      const float q = adam_ratio_fast(m, vv, eps, cert);
      if ((adam_eps_safe(eps) & cert.ok()) == 0u) continue;
      ++safe_n;
      const float ref = adam_ratio_ieee(m, vv, eps);
      if (__float_as_uint(q) != __float_as_uint(ref)) { ++bad; out[2] = __float_as_uint(m); out[3] = __float_as_uint(vv); }
    }
  }
  if (bad) atomicAdd(&out[0], bad);
  if (safe_n) atomicAdd(&out[1], safe_n);
}

// Register-only FMA loop: 16 independent accumulators per thread, `iters` rounds.
__global__ void ffma_peak_kernel(float* out, int iters) {
  float acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0.001f * (float)threadIdx.x + (float)i;
  const float x = 1.0001f, y = 0.5f;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = __fmaf_rn(acc[i], x, y);
  }
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) sum += acc[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = sum;
}

__global__ void debug_exp_kernel(const float* x, int64_t count, float* out) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = spec_expf(x[i]);
}

}  // namespace bbo
