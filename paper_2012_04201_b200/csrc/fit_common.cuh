// Shared definitions of the fit kernels: argument block, shared-memory layout, k-fold
// segments and the in-kernel permutation (sort of Philox keys).  Paper sec. 2 (cross-validation
// score as the evaluated function); the split and shuffling rules are this library's readings.
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
  const float* Xt;       // hold-out mode: test rows [n_test][dp] (null otherwise)
  const float* yt;       // hold-out mode: test labels / targets [n_test]
  int32_t n_test;        // hold-out mode: number of test rows (0 otherwise)
  const Config* configs; // [n_configs]
  const int2* fits;      // this launch's (configuration, fold) list, costliest first
  float* fold_scores;    // [n_configs * K]
  float* trace;          // [n_configs * K * trace_steps] or null
  float* keep_theta;     // parameters of fit (n_configs-1, K-1) in dense layout, or null
  int32_t n_fits, n_configs;
  int32_t config_base;   // added to a configuration's list index when keying its random streams
  const int32_t* config_keys;  // [n_configs] keys of the random streams, replacing index + base (null: unused)
  int32_t n, d, dp, C, CS, K, task;
  int32_t Hs;            // padded hidden width shared by every fit of this launch
  int32_t TB;            // rows per sub-tile (multiple of 4, at most 32)
  int32_t extra_warps;   // pipelined schedule: warps after the tile / unit owners that run the output layer
  int32_t solver;        // 0 Adam, 1 SGD with Nesterov momentum (momentum = beta1)
  int32_t metric;        // 0 accuracy / -MSE, 1 -NLL / -MAE
  int32_t trace_steps, loss_cap;  // loss_cap: rows of the per-row loss buffer
  int32_t order_bytes;   // bytes reserved for the epoch order (uint16 per training row)
  int32_t tmem_cols;     // tensor-memory columns of the CTA (power of two): home of the W1 moments
  uint64_t seed;
};

__host__ __device__ inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

// Shared-memory layout of one fit (float offsets inside a parameter-sized block).  W1 is
// [d][Hs]; W2 is stored transposed, [C][Hs + 4] (class-major, so that the output layer reads
// four consecutive hidden units of one class with one 16-byte load; the pitch of Hs + 4 keeps
// the classes of one load on different banks).  Columns H..Hs+3 of W2 stay zero.
struct Layout {
  int Hs, WP, oW1, ob1, oW2, ob2, PS, PT;
  __host__ __device__ Layout(int d, int Hs_, int C, int CS) {
    Hs = Hs_;
    WP = Hs + 4;           // pitch of a W2 class row, also of an A1 / delta1 row
    oW1 = 0;
    ob1 = d * Hs;
    oW2 = ob1 + Hs;
    ob2 = oW2 + C * WP;
    PS = ob2 + CS;
    PT = PS - ob1;         // everything but W1
  }
};

__host__ __device__ inline int next_pow2(int x) {
  int p = 4;
  while (p < x) p <<= 1;
  return p;
}

// Fold index that keys the random streams of a hold-out fit (no cross-validation fold has it).
constexpr uint32_t kHoldoutFoldKey = 0xFFFFu;

constexpr int kSortBuckets = 2048;  // power of two

// Scratch of the in-kernel permutation: one 64-bit key per element plus the bucket counters.
__host__ __device__ inline size_t sort_scratch_bytes(int n) { return 8u * (size_t)round_up(n, 2) + 4u * kSortBuckets; }

// Dynamic shared memory of one fit (the moments of W1 live in tensor memory, not here).
// pipe: the pipelined schedule (three row buffers, two activation buffers).
__host__ __device__ inline size_t fit_smem_bytes(int d, int dp, int Hs, int C, int CS, int TB, int order_bytes,
                                                 int loss_cap, int n_sort, bool pipe = false) {
  const Layout L(d, Hs, C, CS);
  size_t bytes = 4u * (size_t)(L.PS + 2 * L.PT);
  bytes += (size_t)order_bytes + (size_t)round_up(4 * loss_cap, 16) + (pipe ? 12u : 8u) * TB + 4u * (size_t)TB * CS;
  const size_t xa = (pipe ? 12u : 8u) * (size_t)TB * dp + (pipe ? 8u : 4u) * (size_t)TB * (Hs + 4);
  const size_t keys = sort_scratch_bytes(n_sort);
  return bytes + (xa > keys ? xa : keys);
}

__host__ __device__ inline void fold_segment(int n, int K, int f, int* begin, int* size) {
  const int base = n / K, rem = n % K;
  *begin = f * base + (f < rem ? f : rem);
  *size = base + (f < rem ? 1 : 0);
}

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gmem_src) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }

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

// Permutation of 0..N-1 by ascending (random word << 32 | index), for the fit kernel: the
// words are bucketed by their top bits (counting sort with shared-memory atomics), and each
// bucket, which holds about N / kSortBuckets keys, is ordered by insertion.  The result is the
// unique ascending order of the keys, whatever order the atomics ran in.  scratch:
// sort_scratch_bytes(N) bytes, 8-byte aligned.  The sorted keys are left in keys[0..N); the
// block is synchronised on return.  red: 32 words of shared memory.
__device__ inline uint64_t* bucket_sorted_keys(void* scratch, uint32_t* red, int N, uint64_t seed, uint32_t stream,
                                               uint32_t a, uint32_t b, uint32_t c, int tid, int nt) {
  uint64_t* keys = reinterpret_cast<uint64_t*>(scratch);
  uint32_t* cnt = reinterpret_cast<uint32_t*>(keys + round_up(N, 2));
  constexpr int shift = 32 - 11;
  static_assert(kSortBuckets == (1 << 11), "bucket index uses the top 11 bits");
  const int n_blk = (N + 3) >> 2;
  for (int i = tid; i < kSortBuckets; i += nt) cnt[i] = 0u;
  __syncthreads();
  for (int blk = tid; blk < n_blk; blk += nt) {  // count
    const uint4 r = philox4x32_10(seed, stream, a, b, c, (uint32_t)blk);
#pragma unroll
    for (int w = 0; w < 4; ++w)
      if (4 * blk + w < N) atomicAdd(&cnt[word_of(r, w) >> shift], 1u);
  }
  __syncthreads();
  {  // exclusive scan of the counters, in place
    const int chunk = (kSortBuckets + nt - 1) / nt;
    const int lo = tid * chunk, hi = (lo + chunk) < kSortBuckets ? (lo + chunk) : kSortBuckets;
    uint32_t sum = 0u;
    for (int i = lo; i < hi; ++i) sum += cnt[i];
    uint32_t incl = sum;
    const int lane = tid & 31, warp = tid >> 5;
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += t;
    }
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    uint32_t base = incl - sum;
    for (int w = 0; w < warp; ++w) base += red[w];
    for (int i = lo; i < hi; ++i) { const uint32_t t = cnt[i]; cnt[i] = base; base += t; }
  }
  __syncthreads();
  for (int blk = tid; blk < n_blk; blk += nt) {  // scatter; afterwards cnt[k] = end of bucket k
    const uint4 r = philox4x32_10(seed, stream, a, b, c, (uint32_t)blk);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int i = 4 * blk + w;
      if (i < N) {
        const uint32_t word = word_of(r, w);
        const uint32_t slot = atomicAdd(&cnt[word >> shift], 1u);
        keys[slot] = ((uint64_t)word << 32) | (uint32_t)i;
      }
    }
  }
  __syncthreads();
  for (int k = tid; k < kSortBuckets; k += nt) {  // order each bucket
    const int lo = k == 0 ? 0 : (int)cnt[k - 1], hi = (int)cnt[k];
    for (int i = lo + 1; i < hi; ++i) {
      const uint64_t x = keys[i];
      int j = i - 1;
      while (j >= lo && keys[j] > x) { keys[j + 1] = keys[j]; --j; }
      keys[j + 1] = x;
    }
  }
  __syncthreads();
  return keys;
}

// Dataset row visited i-th in epoch `epoch`: the epoch permutation applied to the training
// list (fold permutation with the held-out segment removed, order kept).
__device__ inline void build_epoch_order(void* scratch, uint32_t* red, uint16_t* order, const int32_t* pi, int n_tr,
                                         int vb, int vs, uint64_t seed, uint32_t config, uint32_t fold,
                                         uint32_t epoch, int tid, int nt) {
  const uint64_t* keys = bucket_sorted_keys(scratch, red, n_tr, seed, kStreamPerm, config, fold, epoch, tid, nt);
  for (int i = tid; i < n_tr; i += nt) {
    const int s = (int)(uint32_t)keys[i];
    order[i] = (uint16_t)pi[s < vb ? s : s + vs];
  }
  __syncthreads();
}

}  // namespace bbo
