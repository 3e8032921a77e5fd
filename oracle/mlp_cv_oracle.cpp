// CPU checker for k-fold cross-validated MLP-Adam evaluation.  TEST INFRASTRUCTURE:
// a plain, slow, single-file reference used only by the tests, the smoke check and the
// benchmark's CPU-baseline leg.  It shares no code with the CUDA library and the CUDA
// library never calls it.
//
// What it computes (paper sec. 2: the function a black-box optimizer sees is "the cross
// validation score of a machine learning model on a dataset with a loss function";
// Algorithm 1: scores = evaluate(params_list); Table 1: model MLP-adam, metrics acc / mse;
// sec. 6.3: 2.7 M trainings / 541,440 evaluations = 5 folds).  The paper gives no formula
// for the model; the readings taken here are the scikit-learn MLP it names: one hidden
// ReLU layer, softmax cross-entropy (classification) or half mean squared error
// (regression), L2 penalty alpha/(2*batch) on the weight matrices, Adam in the
// Kingma-Ba "efficient" form, Glorot-uniform initialisation, shuffled minibatches each
// epoch.  Every floating-point operation on the training path has a fixed order so that
// the float mode is reproducible bit for bit; the double mode runs the same steps in
// binary64 and exists for gradient checks and distance-from-truth reports.  Three further modes
// are experiments, never references; they ask what tensor-core arithmetic in the two large
// contractions (X W1 and X^T delta1) would do to the scores, everything else staying float:
// operands rounded to TF32; float products summed the way a matrix unit sums them (blocks of
// eight terms, block sums added in order); and that blocking with every operand split into a
// TF32 high and low part and three products per term.
//
// Pinned (tests/test_oracle_*.py) against: the published Philox-4x32-10 known answers, a
// Python big-integer restatement and the inverse bijection; libm exp; torch autograd
// gradients and central finite differences; torch.optim.Adam and the first-step closed
// form; scikit-learn's own MLPClassifier/MLPRegressor partial_fit steps; brute-force
// rescoring from the final weights; least-squares and separable-data limits.
//
// Build: g++ -O2 -ffp-contract=off -mfma -fopenmp -shared -fPIC mlp_cv_oracle.cpp
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------
// Counter-based random numbers: Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11).  key = the 64-bit seed,
// counter = (blk, a, b, stream << 28 | c).  Element i of a draw is word i&3 of block i>>2.
// ---------------------------------------------------------------------------------------
enum : uint32_t { STREAM_FOLD = 1, STREAM_INIT = 2, STREAM_PERM = 3 };

void philox_block(uint64_t seed, uint32_t stream, uint32_t a, uint32_t b, uint32_t c, uint32_t blk,
                  uint32_t out[4]) {
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
  uint32_t x0 = blk, x1 = a, x2 = b, x3 = (stream << 28) | (c & 0x0FFFFFFFu);
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * x0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * x2;
    uint32_t y0 = (uint32_t)(p1 >> 32) ^ x1 ^ k0;
    uint32_t y1 = (uint32_t)p1;
    uint32_t y2 = (uint32_t)(p0 >> 32) ^ x3 ^ k1;
    uint32_t y3 = (uint32_t)p0;
    x0 = y0; x1 = y1; x2 = y2; x3 = y3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = x0; out[1] = x1; out[2] = x2; out[3] = x3;
}

uint32_t rng_word(uint64_t seed, uint32_t stream, uint32_t a, uint32_t b, uint32_t c, uint32_t i) {
  uint32_t w[4];
  philox_block(seed, stream, a, b, c, i >> 2, w);
  return w[i & 3];
}

// Permutation of 0..N-1: sort indices by the 64-bit key (random word << 32 | index).
void rng_perm(int32_t N, uint64_t seed, uint32_t stream, uint32_t a, uint32_t b, uint32_t c,
              std::vector<int32_t>& out) {
  std::vector<uint64_t> key((size_t)N);
  for (int32_t i = 0; i < N; ++i)
    key[i] = ((uint64_t)rng_word(seed, stream, a, b, c, (uint32_t)i) << 32) | (uint32_t)i;
  std::sort(key.begin(), key.end());
  out.resize((size_t)N);
  for (int32_t i = 0; i < N; ++i) out[i] = (int32_t)(key[i] & 0xFFFFFFFFu);
}

// Shuffled, non-stratified K-fold: one permutation pi of the rows per (seed, n); fold f is
// a contiguous segment of pi, the first n mod K folds one row longer.
void fold_segment(int64_t n, int32_t K, int32_t f, int64_t* begin, int64_t* size) {
  int64_t base = n / K, rem = n % K;
  *begin = (int64_t)f * base + std::min<int64_t>(f, rem);
  *size = base + (f < rem ? 1 : 0);
}

// ---------------------------------------------------------------------------------------
// The float exponential used by the softmax.  Fixed sequence of IEEE operations so that any
// implementation following it returns the same bits: n = rint(x*log2(e)); r = x - n*ln2 in
// two fused steps; degree-7 Taylor polynomial by Horner with fused multiply-adds; scale by
// 2^n through the exponent field.
// ---------------------------------------------------------------------------------------
float spec_expf(float x) {
  if (x != x) return x;
  if (x < -86.0f) return 0.0f;
  if (x > 88.0f) return std::numeric_limits<float>::infinity();
  float t = x * 0x1.715476p+0f;          // log2(e) rounded to float
  float n = std::nearbyintf(t);          // round to nearest, ties to even
  float r = std::fmaf(n, -0x1.62e4p-1f, x);       // ln2 high part (0x3F317200)
  r = std::fmaf(n, -0x1.7f7d1cp-20f, r);          // ln2 low part  (0x35BFBE8E)
  float p = 0x1.a01a02p-13f;             // 1/5040
  p = std::fmaf(p, r, 0x1.6c16c2p-10f);  // 1/720
  p = std::fmaf(p, r, 0x1.111112p-7f);   // 1/120
  p = std::fmaf(p, r, 0x1.555556p-5f);   // 1/24
  p = std::fmaf(p, r, 0x1.555556p-3f);   // 1/6
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  int32_t e = (int32_t)n + 127;          // 3 <= e <= 254 on the admitted range
  uint32_t bits = (uint32_t)e << 23;
  float scale;
  std::memcpy(&scale, &bits, 4);
  return p * scale;
}

template <typename T> struct Fn;
template <> struct Fn<float> {
  static float exp_(float x) { return spec_expf(x); }
  static float log_(float x) { return std::log(x); }
  static float sqrt_(float x) { return std::sqrt(x); }
  static float fma_(float a, float b, float c) { return std::fmaf(a, b, c); }
};
template <> struct Fn<double> {
  static double exp_(double x) { return std::exp(x); }
  static double log_(double x) { return std::log(x); }
  static double sqrt_(double x) { return std::sqrt(x); }
  static double fma_(double a, double b, double c) { return std::fma(a, b, c); }
};

// Round-to-nearest-even to the 10-bit mantissa of the TF32 tensor-core input format (inf and NaN
// pass through).  Used only by the experiment mode that asks what such operands would do to the
// scores; the products are still accumulated in the mode's own precision.
inline float tf32_round(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if (((u >> 23) & 0xFFu) == 0xFFu) return x;
  u += 0xFFFu + ((u >> 13) & 1u);
  u &= ~0x1FFFu;
  float y;
  std::memcpy(&y, &u, 4);
  return y;
}
template <typename T> inline T tf32_operand(T x) { return (T)tf32_round((float)x); }

// Experiment modes of the two large contractions (Shape::exp).
enum : int32_t {
  EXP_NONE = 0,
  EXP_TF32_OPERANDS = 2,  // operands rounded to TF32, terms added one by one in the usual order
  EXP_BLOCKED = 3,        // exact float products; terms in blocks of 8 summed from zero, block sums added in order
  EXP_BLOCKED_SPLIT = 4   // EXP_BLOCKED with each operand split hi + lo (both TF32) and lo*hi + hi*lo + hi*hi per term
};
constexpr int32_t kMmaBlock = 8;

// hi = tf32(x), lo = tf32(x - hi): x = hi + lo up to about 2^-21 relative.
inline void tf32_split(float x, float* hi, float* lo) {
  *hi = tf32_round(x);
  *lo = tf32_round(x - *hi);
}

// One term a*b added to the block sum `acc` under an experiment mode.
template <typename T> inline T exp_term(int32_t exp, T a, T b, T acc) {
  if (exp == EXP_BLOCKED_SPLIT) {
    float ah, al, bh, bl;
    tf32_split((float)a, &ah, &al);
    tf32_split((float)b, &bh, &bl);
    acc = Fn<T>::fma_((T)al, (T)bh, acc);
    acc = Fn<T>::fma_((T)ah, (T)bl, acc);
    return Fn<T>::fma_((T)ah, (T)bh, acc);
  }
  return Fn<T>::fma_(a, b, acc);
}

struct Config {  // one suggested configuration, 32 bytes; same field order as the library's
  int32_t hidden, batch_size, epochs;
  float alpha, lr, beta1, beta2, eps;
};

// Parameter vector layout: W1[d][H] row-major, b1[H], W2[H][C] row-major, b2[C].
struct Shape {
  int32_t d, H, C;
  int32_t exp = EXP_NONE;  // experiment mode of the two large contractions (never a reference)
  int64_t oW1() const { return 0; }
  int64_t ob1() const { return (int64_t)d * H; }
  int64_t oW2() const { return ob1() + H; }
  int64_t ob2() const { return oW2() + (int64_t)H * C; }
  int64_t P() const { return ob2() + C; }
};

// Glorot-uniform for weights and biases of a layer: bound = sqrt(6/(fan_in+fan_out)),
// value = bound * (2u - 1), u = (word >> 8) * 2^-24.  Layer tags: W1=0, b1=1, W2=2, b2=3.
template <typename T>
void init_params(const Shape& s, uint64_t seed, uint32_t config, uint32_t fold, T* th) {
  auto draw = [&](uint32_t layer, uint32_t idx, float bound) -> T {
    uint32_t w = rng_word(seed, STREAM_INIT, config, fold, layer, idx);
    float u = (float)(w >> 8) * 0x1p-24f;
    float v = bound * (2.0f * u - 1.0f);
    return (T)v;
  };
  float bound1 = std::sqrt(6.0f / (float)(s.d + s.H));
  float bound2 = std::sqrt(6.0f / (float)(s.H + s.C));
  for (int64_t i = 0; i < (int64_t)s.d * s.H; ++i) th[s.oW1() + i] = draw(0, (uint32_t)i, bound1);
  for (int32_t j = 0; j < s.H; ++j) th[s.ob1() + j] = draw(1, (uint32_t)j, bound1);
  for (int64_t i = 0; i < (int64_t)s.H * s.C; ++i) th[s.oW2() + i] = draw(2, (uint32_t)i, bound2);
  for (int32_t o = 0; o < s.C; ++o) th[s.ob2() + o] = draw(3, (uint32_t)o, bound2);
}

// Forward pass for one row: z1 (pre-activation), a1 (ReLU), z2 (output).
template <typename T>
void forward_row(const Shape& s, const T* th, const T* x, T* z1, T* a1, T* z2) {
  const T* W1 = th + s.oW1(); const T* b1 = th + s.ob1();
  const T* W2 = th + s.oW2(); const T* b2 = th + s.ob2();
  // z1[j] = b1[j] + sum_k x[k] W1[k][j], each sum accumulated in ascending k by fused
  // multiply-add (the k loop is outermost only so that memory is walked row by row).
  for (int32_t j = 0; j < s.H; ++j) z1[j] = b1[j];
  if (s.exp == EXP_TF32_OPERANDS) {
    for (int32_t k = 0; k < s.d; ++k)
      for (int32_t j = 0; j < s.H; ++j)
        z1[j] = Fn<T>::fma_(tf32_operand(x[k]), tf32_operand(W1[(int64_t)k * s.H + j]), z1[j]);
  } else if (s.exp == EXP_BLOCKED || s.exp == EXP_BLOCKED_SPLIT) {
    for (int32_t j = 0; j < s.H; ++j)
      for (int32_t k0 = 0; k0 < s.d; k0 += kMmaBlock) {
        T part = (T)0;
        for (int32_t k = k0; k < s.d && k < k0 + kMmaBlock; ++k) part = exp_term<T>(s.exp, x[k], W1[(int64_t)k * s.H + j], part);
        z1[j] = z1[j] + part;
      }
  } else {
    for (int32_t k = 0; k < s.d; ++k)
      for (int32_t j = 0; j < s.H; ++j) z1[j] = Fn<T>::fma_(x[k], W1[(int64_t)k * s.H + j], z1[j]);
  }
  for (int32_t j = 0; j < s.H; ++j) a1[j] = z1[j] > (T)0 ? z1[j] : (T)0;
  // z2[o] = b2[o] + sum_j a1[j] W2[j][o], ascending j.
  for (int32_t o = 0; o < s.C; ++o) z2[o] = b2[o];
  for (int32_t j = 0; j < s.H; ++j)
    for (int32_t o = 0; o < s.C; ++o) z2[o] = Fn<T>::fma_(a1[j], W2[(int64_t)j * s.C + o], z2[o]);
}

// Minibatch loss and gradient (L2 term included in both).  xb: Bs rows of d values, yb: Bs
// labels/targets.  task 0: softmax cross-entropy, mean over the batch; task 1: half mean
// squared error.  Penalty alpha/(2 Bs) (|W1|^2 + |W2|^2), biases unpenalised.
// All sums over the batch run in ascending row order; all sums over k, j, o ascending.
template <typename T>
T loss_and_grad(const Shape& s, int32_t task, T alpha, const T* th, const T* xb, const T* yb,
                int32_t Bs, T* grad, bool want_loss) {
  const int32_t d = s.d, H = s.H, C = s.C;
  const T* W1 = th + s.oW1(); const T* W2 = th + s.oW2();
  std::vector<T> z1((size_t)Bs * H), a1((size_t)Bs * H), z2((size_t)Bs * C), d2((size_t)Bs * C),
      d1((size_t)Bs * H);
  const T invB = (T)1 / (T)Bs;
  T loss_sum = (T)0;
  for (int32_t b = 0; b < Bs; ++b) {
    forward_row(s, th, xb + (int64_t)b * d, &z1[(size_t)b * H], &a1[(size_t)b * H], &z2[(size_t)b * C]);
    const T* z = &z2[(size_t)b * C];
    T* dl = &d2[(size_t)b * C];
    if (task == 0) {
      int32_t label = (int32_t)yb[b];
      T mx = z[0];
      for (int32_t o = 1; o < C; ++o) if (z[o] > mx) mx = z[o];
      T sum = (T)0;
      for (int32_t o = 0; o < C; ++o) { dl[o] = Fn<T>::exp_(z[o] - mx); sum = sum + dl[o]; }
      for (int32_t o = 0; o < C; ++o) {
        T p = dl[o] / sum;
        dl[o] = (p - (o == label ? (T)1 : (T)0)) * invB;
      }
      if (want_loss) loss_sum = loss_sum + (Fn<T>::log_(sum) - (z[label] - mx));
    } else {
      T r = z[0] - yb[b];
      dl[0] = r * invB;
      if (want_loss) loss_sum = loss_sum + (T)0.5 * r * r;
    }
  }
  T* gW1 = grad + s.oW1(); T* gb1 = grad + s.ob1(); T* gW2 = grad + s.oW2(); T* gb2 = grad + s.ob2();
  // gW2[j][o] = sum_b a1[b][j] d2[b][o], every sum in ascending b (b outermost: row-wise walk).
  for (int64_t i = 0; i < (int64_t)H * C; ++i) gW2[i] = (T)0;
  for (int32_t b = 0; b < Bs; ++b)
    for (int32_t j = 0; j < H; ++j)
      for (int32_t o = 0; o < C; ++o)
        gW2[(int64_t)j * C + o] = Fn<T>::fma_(a1[(size_t)b * H + j], d2[(size_t)b * C + o], gW2[(int64_t)j * C + o]);
  for (int32_t o = 0; o < C; ++o) {
    T acc = (T)0;
    for (int32_t b = 0; b < Bs; ++b) acc = acc + d2[(size_t)b * C + o];
    gb2[o] = acc;
  }
  for (int32_t b = 0; b < Bs; ++b)
    for (int32_t j = 0; j < H; ++j) {
      T acc = (T)0;
      for (int32_t o = 0; o < C; ++o) acc = Fn<T>::fma_(d2[(size_t)b * C + o], W2[(int64_t)j * C + o], acc);
      d1[(size_t)b * H + j] = z1[(size_t)b * H + j] > (T)0 ? acc : (T)0;
    }
  // gW1[k][j] = sum_b x[b][k] d1[b][j], every sum in ascending b.
  for (int64_t i = 0; i < (int64_t)d * H; ++i) gW1[i] = (T)0;
  if (s.exp == EXP_TF32_OPERANDS) {
    for (int32_t b = 0; b < Bs; ++b)
      for (int32_t k = 0; k < d; ++k)
        for (int32_t j = 0; j < H; ++j)
          gW1[(int64_t)k * H + j] = Fn<T>::fma_(tf32_operand(xb[(int64_t)b * d + k]), tf32_operand(d1[(size_t)b * H + j]),
                                                gW1[(int64_t)k * H + j]);
  } else if (s.exp == EXP_BLOCKED || s.exp == EXP_BLOCKED_SPLIT) {
    for (int32_t k = 0; k < d; ++k)
      for (int32_t j = 0; j < H; ++j) {
        T acc = (T)0;
        for (int32_t b0 = 0; b0 < Bs; b0 += kMmaBlock) {
          T part = (T)0;
          for (int32_t b = b0; b < Bs && b < b0 + kMmaBlock; ++b)
            part = exp_term<T>(s.exp, xb[(int64_t)b * d + k], d1[(size_t)b * H + j], part);
          acc = acc + part;
        }
        gW1[(int64_t)k * H + j] = acc;
      }
  } else {
    for (int32_t b = 0; b < Bs; ++b)
      for (int32_t k = 0; k < d; ++k)
        for (int32_t j = 0; j < H; ++j)
          gW1[(int64_t)k * H + j] = Fn<T>::fma_(xb[(int64_t)b * d + k], d1[(size_t)b * H + j], gW1[(int64_t)k * H + j]);
  }
  for (int32_t j = 0; j < H; ++j) {
    T acc = (T)0;
    for (int32_t b = 0; b < Bs; ++b) acc = acc + d1[(size_t)b * H + j];
    gb1[j] = acc;
  }
  // L2 penalty gradient on the weight matrices, with the weights of before the update.
  const T aB = alpha * invB;
  for (int64_t i = 0; i < (int64_t)d * H; ++i) gW1[i] = Fn<T>::fma_(aB, W1[i], gW1[i]);
  for (int64_t i = 0; i < (int64_t)H * C; ++i) gW2[i] = Fn<T>::fma_(aB, W2[i], gW2[i]);
  if (!want_loss) return (T)0;
  T sq = (T)0;
  for (int64_t i = 0; i < (int64_t)d * H; ++i) sq = Fn<T>::fma_(W1[i], W1[i], sq);
  for (int64_t i = 0; i < (int64_t)H * C; ++i) sq = Fn<T>::fma_(W2[i], W2[i], sq);
  return loss_sum * invB + ((T)0.5 * alpha * invB) * sq;
}

// Adam (Kingma & Ba 2015, the form with the bias corrections folded into the step size):
// step_t = lr sqrt(1 - beta2^t) / (1 - beta1^t); theta -= step_t * m / (sqrt(v) + eps).
// beta^t are running products in double; step_t is rounded to T once per step.
template <typename T>
struct Adam {
  T lr, beta1, beta2, eps;
  double p1 = 1.0, p2 = 1.0;
  int64_t t = 0;
  void update(int64_t P, T* th, T* m, T* v, const T* g) {
    t += 1;
    p1 *= (double)beta1;
    p2 *= (double)beta2;
    const T step = (T)((double)lr * std::sqrt(1.0 - p2) / (1.0 - p1));
    const T omb1 = (T)1 - beta1, omb2 = (T)1 - beta2;
    for (int64_t i = 0; i < P; ++i) {
      m[i] = Fn<T>::fma_(beta1, m[i], omb1 * g[i]);
      v[i] = Fn<T>::fma_(beta2, v[i], (omb2 * g[i]) * g[i]);
      th[i] = th[i] - step * (m[i] / (Fn<T>::sqrt_(v[i]) + eps));
    }
  }
};

// Stochastic gradient descent with Nesterov momentum (the paper's Table 1 lists MLP-sgd beside
// MLP-adam; this is the update of the scikit-learn solver it names, constant learning rate):
// velocity = momentum * velocity - lr * g; theta += momentum * velocity - lr * g, the second
// expression taken with the new velocity.  lr * g is rounded once and used in both; each of the
// two expressions is one fused multiply-add.
template <typename T>
struct Sgd {
  T lr, momentum;
  void update(int64_t P, T* th, T* vel, const T* g) {
    for (int64_t i = 0; i < P; ++i) {
      const T t = lr * g[i];
      vel[i] = Fn<T>::fma_(momentum, vel[i], -t);
      th[i] = th[i] + Fn<T>::fma_(momentum, vel[i], -t);
    }
  }
};

enum : int32_t { SOLVER_ADAM = 0, SOLVER_SGD = 1 };
enum : int32_t { METRIC_DEFAULT = 0, METRIC_ALT = 1 };  // accuracy / -MSE, or -NLL / -MAE (Table 1: nll, mae)

// Held-out score of one fit: accuracy (prediction = lowest index attaining the maximum
// under strict >, so a NaN never wins) or negative mean squared error (NaN -> -inf).
template <typename T>
T score_rows(const Shape& s, int32_t task, int32_t metric, const T* th, const float* X, const float* y,
             const int32_t* rows, int32_t n_rows) {
  std::vector<T> x((size_t)s.d), z1((size_t)s.H), a1((size_t)s.H), z2((size_t)s.C);
  int32_t correct = 0;
  T sq = (T)0;
  for (int32_t i = 0; i < n_rows; ++i) {
    const float* xr = X + (int64_t)rows[i] * s.d;
    for (int32_t k = 0; k < s.d; ++k) x[k] = (T)xr[k];
    forward_row(s, th, x.data(), z1.data(), a1.data(), z2.data());
    if (task == 0 && metric == METRIC_ALT) {
      // negative log-likelihood of the true class under the softmax (same max-subtraction,
      // exponential and ascending denominator as in training), summed over rows in order
      const int32_t label = (int32_t)y[rows[i]];
      T mx = z2[0];
      for (int32_t o = 1; o < s.C; ++o) if (z2[o] > mx) mx = z2[o];
      T sum = (T)0;
      for (int32_t o = 0; o < s.C; ++o) sum = sum + Fn<T>::exp_(z2[o] - mx);
      sq = sq + (Fn<T>::log_(sum) - (z2[label] - mx));
    } else if (task == 0) {
      int32_t best = 0;
      for (int32_t o = 1; o < s.C; ++o) if (z2[o] > z2[best]) best = o;
      if (best == (int32_t)y[rows[i]]) ++correct;
    } else if (metric == METRIC_ALT) {
      T r = z2[0] - (T)y[rows[i]];
      sq = sq + (r < (T)0 ? -r : r);
    } else {
      T r = z2[0] - (T)y[rows[i]];
      sq = Fn<T>::fma_(r, r, sq);
    }
  }
  if (task == 0 && metric == METRIC_DEFAULT) return (T)correct / (T)n_rows;
  T s_ = -(sq / (T)n_rows);
  if (s_ != s_) s_ = -std::numeric_limits<T>::infinity();
  return s_;
}

// One (config, fold) fit: split, initialise, train E epochs, score the held-out fold.
// trace (may be null): per-step training loss of the first trace_steps optimizer steps,
// NaN-padded when the fit has fewer steps.  theta_out (may be null): final parameters.
template <typename T>
double run_fit(const float* X, const float* y, int64_t n, int32_t d, int32_t C, int32_t task,
               int32_t K, const Config& cf, uint32_t config, uint32_t fold, uint64_t seed,
               const std::vector<int32_t>& pi, int32_t trace_steps, double* trace, double* theta_out,
               int32_t solver = SOLVER_ADAM, int32_t metric = METRIC_DEFAULT, const float* Xtest = nullptr,
               const float* ytest = nullptr, int64_t n_test = 0, int32_t exp = EXP_NONE) {
  // Hold-out mode (Xtest given; paper sec. 6.2: the generalisation score is taken on data held
  // out from the optimisation): train on every row, in the order of the fold permutation, and
  // score the rows of (Xtest, ytest) in their own order.  `fold` then only keys the random streams.
  int64_t vb = 0, vs = 0;
  if (!Xtest) fold_segment(n, K, (int32_t)fold, &vb, &vs);
  std::vector<int32_t> val(pi.begin() + vb, pi.begin() + vb + vs), train;
  train.reserve((size_t)(n - vs));
  for (int64_t i = 0; i < n; ++i) if (i < vb || i >= vb + vs) train.push_back(pi[i]);
  if (Xtest) { val.resize((size_t)n_test); for (int64_t i = 0; i < n_test; ++i) val[(size_t)i] = (int32_t)i; }
  const int32_t n_tr = (int32_t)train.size();
  const int32_t B = std::min(cf.batch_size, n_tr);
  Shape s{d, cf.hidden, C};
  s.exp = exp;
  const int64_t P = s.P();
  std::vector<T> th((size_t)P), m((size_t)P, (T)0), v((size_t)P, (T)0), g((size_t)P);
  init_params<T>(s, seed, config, fold, th.data());
  Adam<T> adam{(T)cf.lr, (T)cf.beta1, (T)cf.beta2, (T)cf.eps};
  Sgd<T> sgd{(T)cf.lr, (T)cf.beta1};  // beta1 doubles as the momentum
  std::vector<T> xb((size_t)B * d), yb((size_t)B);
  std::vector<int32_t> sigma;
  for (int32_t i = 0; i < trace_steps; ++i) if (trace) trace[i] = std::numeric_limits<double>::quiet_NaN();
  int64_t step_no = 0;
  for (int32_t e = 0; e < cf.epochs; ++e) {
    rng_perm(n_tr, seed, STREAM_PERM, config, fold, (uint32_t)e, sigma);
    for (int32_t s0 = 0; s0 < n_tr; s0 += B) {
      const int32_t Bs = std::min(B, n_tr - s0);
      for (int32_t b = 0; b < Bs; ++b) {
        const int32_t row = train[sigma[s0 + b]];
        for (int32_t k = 0; k < d; ++k) xb[(size_t)b * d + k] = (T)X[(int64_t)row * d + k];
        yb[b] = (T)y[row];
      }
      const bool want = trace && step_no < trace_steps;
      T loss = loss_and_grad<T>(s, task, (T)cf.alpha, th.data(), xb.data(), yb.data(), Bs, g.data(), want);
      if (want) trace[step_no] = (double)loss;
      if (solver == SOLVER_SGD) sgd.update(P, th.data(), m.data(), g.data());
      else adam.update(P, th.data(), m.data(), v.data(), g.data());
      ++step_no;
    }
  }
  if (theta_out) for (int64_t i = 0; i < P; ++i) theta_out[i] = (double)th[i];
  return (double)score_rows<T>(s, task, metric, th.data(), Xtest ? Xtest : X, Xtest ? ytest : y, val.data(),
                               (int32_t)val.size());
}

int validate(const float* X, const float* y, int64_t n, int32_t d, int32_t task, int32_t K,
             const Config* cfg, int32_t n_configs) {
  if (!X || !y || !cfg || n < 2 || d < 1 || K < 2 || K > n || n_configs < 0) return -1;
  if (task != 0 && task != 1) return -1;
  for (int32_t c = 0; c < n_configs; ++c) {
    const Config& q = cfg[c];
    if (q.hidden < 1 || q.batch_size < 1 || q.epochs < 0 || q.epochs >= (1 << 28)) return -1;
    if (!(q.alpha >= 0.f) || !(q.lr >= 0.f) || !(q.beta1 >= 0.f && q.beta1 < 1.f) ||
        !(q.beta2 >= 0.f && q.beta2 < 1.f) || !(q.eps > 0.f))
      return -1;
  }
  return 0;
}

int derive_classes(const float* y, int64_t n, int32_t task, int32_t n_classes) {
  if (task == 1) return 1;
  int32_t mx = 0;
  for (int64_t i = 0; i < n; ++i) {
    float v = y[i];
    if (!(v >= 0.f) || v != std::floor(v) || v > 1e6f) return -1;
    mx = std::max(mx, (int32_t)v);
  }
  if (n_classes > 0) return mx < n_classes ? n_classes : -1;
  return mx + 1;
}

}  // namespace

extern "C" {

void oracle_rng_block(uint64_t seed, uint32_t stream, uint32_t a, uint32_t b, uint32_t c, uint32_t blk,
                      uint32_t* out4) {
  philox_block(seed, stream, a, b, c, blk, out4);
}

// Raw Philox-4x32-10 on an arbitrary counter/key (for the published known answers).
void oracle_philox_raw(const uint32_t* ctr4, const uint32_t* key2, uint32_t* out4) {
  uint64_t seed = (uint64_t)key2[0] | ((uint64_t)key2[1] << 32);
  // counter words map as (blk, a, b, word3); pass word3 through stream/c split
  philox_block(seed, ctr4[3] >> 28, ctr4[1], ctr4[2], ctr4[3] & 0x0FFFFFFFu, ctr4[0], out4);
}

void oracle_perm(int32_t N, uint64_t seed, uint32_t stream, uint32_t a, uint32_t b, uint32_t c, int32_t* out) {
  std::vector<int32_t> p;
  rng_perm(N, seed, stream, a, b, c, p);
  std::copy(p.begin(), p.end(), out);
}

// fold_of_row[n]: fold each row is held out in.  pi[n]: the fold permutation.
int oracle_fold_split(int64_t n, int32_t K, uint64_t seed, int32_t* pi_out, int32_t* fold_of_row) {
  if (n < 2 || K < 2 || K > n) return -1;
  std::vector<int32_t> pi;
  rng_perm((int32_t)n, seed, STREAM_FOLD, 0, 0, 0, pi);
  for (int32_t f = 0; f < K; ++f) {
    int64_t b, s;
    fold_segment(n, K, f, &b, &s);
    for (int64_t i = b; i < b + s; ++i) fold_of_row[pi[i]] = f;
  }
  if (pi_out) std::copy(pi.begin(), pi.end(), pi_out);
  return 0;
}

// Row order of one epoch of one fit: order[i] = dataset row of the i-th training sample
// visited in epoch `epoch`.  Returns n_train (or -1).
int oracle_epoch_order(int64_t n, int32_t K, uint64_t seed, int32_t config, int32_t fold, int32_t epoch,
                       int32_t* order) {
  if (n < 2 || K < 2 || K > n || fold < 0 || fold >= K) return -1;
  std::vector<int32_t> pi, sigma, train;
  rng_perm((int32_t)n, seed, STREAM_FOLD, 0, 0, 0, pi);
  int64_t vb, vs;
  fold_segment(n, K, fold, &vb, &vs);
  for (int64_t i = 0; i < n; ++i) if (i < vb || i >= vb + vs) train.push_back(pi[i]);
  rng_perm((int32_t)train.size(), seed, STREAM_PERM, (uint32_t)config, (uint32_t)fold, (uint32_t)epoch, sigma);
  for (size_t i = 0; i < train.size(); ++i) order[i] = train[sigma[i]];
  return (int)train.size();
}

float oracle_expf(float x) { return spec_expf(x); }

void oracle_expf_array(const float* x, int64_t count, float* out) {
  for (int64_t i = 0; i < count; ++i) out[i] = spec_expf(x[i]);
}

// counters[count][5] = (stream, a, b, c, blk) -> out[count][4]
void oracle_rng_blocks(uint64_t seed, const uint32_t* counters, int64_t count, uint32_t* out) {
  for (int64_t i = 0; i < count; ++i)
    philox_block(seed, counters[5 * i], counters[5 * i + 1], counters[5 * i + 2], counters[5 * i + 3],
                 counters[5 * i + 4], out + 4 * i);
}

int64_t oracle_param_count(int32_t d, int32_t H, int32_t C) { return Shape{d, H, C}.P(); }

void oracle_init_params(int32_t d, int32_t H, int32_t C, uint64_t seed, int32_t config, int32_t fold,
                        double* theta) {
  Shape s{d, H, C};
  std::vector<float> th((size_t)s.P());
  init_params<float>(s, seed, (uint32_t)config, (uint32_t)fold, th.data());
  for (int64_t i = 0; i < s.P(); ++i) theta[i] = th[i];
}

// Loss and gradient of one minibatch at given parameters.  mode 0: float arithmetic,
// mode 1: double.  Arrays cross the boundary as double (floats are exact in double).
double oracle_loss_grad(int32_t mode, int32_t d, int32_t H, int32_t C, int32_t task, double alpha,
                        const double* theta, const double* xb, const double* yb, int32_t Bs, double* grad) {
  Shape s{d, H, C};
  const int64_t P = s.P();
  if (mode == 1) return loss_and_grad<double>(s, task, alpha, theta, xb, yb, Bs, grad, true);
  std::vector<float> th(theta, theta + P), x(xb, xb + (int64_t)Bs * d), y(yb, yb + Bs), g((size_t)P);
  float l = loss_and_grad<float>(s, task, (float)alpha, th.data(), x.data(), y.data(), Bs, g.data(), true);
  for (int64_t i = 0; i < P; ++i) grad[i] = g[i];
  return l;
}

// n_steps Adam updates on P parameters with caller-supplied gradients grads[n_steps][P].
void oracle_adam_steps(int32_t mode, int64_t P, int32_t n_steps, double lr, double beta1, double beta2,
                       double eps, double* theta, double* m, double* v, const double* grads) {
  if (mode == 1) {
    Adam<double> a{lr, beta1, beta2, eps};
    for (int32_t s = 0; s < n_steps; ++s) a.update(P, theta, m, v, grads + (int64_t)s * P);
    return;
  }
  std::vector<float> th(theta, theta + P), mm(m, m + P), vv(v, v + P), g((size_t)P);
  Adam<float> a{(float)lr, (float)beta1, (float)beta2, (float)eps};
  for (int32_t s = 0; s < n_steps; ++s) {
    for (int64_t i = 0; i < P; ++i) g[i] = (float)grads[(int64_t)s * P + i];
    a.update(P, th.data(), mm.data(), vv.data(), g.data());
  }
  for (int64_t i = 0; i < P; ++i) { theta[i] = th[i]; m[i] = mm[i]; v[i] = vv[i]; }
}

// A list of (config, fold) fits.  Host pointers throughout.
//   fit_config[n_fits], fit_fold[n_fits]: which fits to run (config index into configs[]).
//   fit_scores[n_fits]; loss_trace[n_fits*trace_steps] (or null); theta_out: parameters of
//   the LAST listed fit (or null).  n_threads <= 0: all cores; threads split fits only.
// mode: 0 float, 1 double; 2, 3, 4: the float experiment modes EXP_TF32_OPERANDS, EXP_BLOCKED,
// EXP_BLOCKED_SPLIT of the two large contractions (X W1 and
// X^T delta1) -- experiment modes that show what tensor-core arithmetic would
// do to the scores; never the reference for anything.
// solver: 0 Adam, 1 SGD with Nesterov momentum (momentum = the configuration's beta1).
// metric: 0 accuracy / -MSE, 1 -NLL / -MAE.
int oracle_mlp_cv_fits_ex(int32_t mode, const float* X, const float* y, int64_t n, int32_t d, int32_t task,
                          int32_t n_folds, const void* configs, int32_t n_configs, uint64_t seed,
                          int32_t n_classes, const int32_t* fit_config, const int32_t* fit_fold, int32_t n_fits,
                          int32_t trace_steps, int32_t n_threads, double* fit_scores, double* loss_trace,
                          double* theta_out, int32_t solver, int32_t metric) {
  if (solver < 0 || solver > 1 || metric < 0 || metric > 1) return -1;
  const Config* cfg = (const Config*)configs;
  if (validate(X, y, n, d, task, n_folds, cfg, n_configs) != 0) return -1;
  const int32_t C = derive_classes(y, n, task, n_classes);
  if (C < 1) return -1;
  for (int32_t i = 0; i < n_fits; ++i)
    if (fit_config[i] < 0 || fit_config[i] >= n_configs || fit_fold[i] < 0 || fit_fold[i] >= n_folds) return -1;
  std::vector<int32_t> pi;
  rng_perm((int32_t)n, seed, STREAM_FOLD, 0, 0, 0, pi);
#ifdef _OPENMP
  if (n_threads <= 0) n_threads = omp_get_num_procs();
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads)
#endif
  for (int32_t i = 0; i < n_fits; ++i) {
    double* tr = loss_trace ? loss_trace + (int64_t)i * trace_steps : nullptr;
    double* tho = (theta_out && i == n_fits - 1) ? theta_out : nullptr;
    const Config& cf = cfg[fit_config[i]];
    fit_scores[i] = mode == 1
        ? run_fit<double>(X, y, n, d, C, task, n_folds, cf, fit_config[i], fit_fold[i], seed, pi, trace_steps, tr, tho, solver, metric)
        : run_fit<float>(X, y, n, d, C, task, n_folds, cf, fit_config[i], fit_fold[i], seed, pi, trace_steps, tr, tho, solver, metric,
                         nullptr, nullptr, 0, /*exp=*/mode >= 2 ? mode : EXP_NONE);
  }
  return 0;
}

int oracle_mlp_cv_fits(int32_t mode, const float* X, const float* y, int64_t n, int32_t d, int32_t task,
                       int32_t n_folds, const void* configs, int32_t n_configs, uint64_t seed,
                       int32_t n_classes, const int32_t* fit_config, const int32_t* fit_fold, int32_t n_fits,
                       int32_t trace_steps, int32_t n_threads, double* fit_scores, double* loss_trace,
                       double* theta_out) {
  return oracle_mlp_cv_fits_ex(mode, X, y, n, d, task, n_folds, configs, n_configs, seed, n_classes, fit_config,
                               fit_fold, n_fits, trace_steps, n_threads, fit_scores, loss_trace, theta_out, 0, 0);
}

// scores = evaluate(params_list): every config, every fold, mean over folds (ascending fold,
// in the mode's precision).  fold_scores[n_configs*n_folds] and loss_trace may be null.
int oracle_mlp_cv_eval_ex(int32_t mode, const float* X, const float* y, int64_t n, int32_t d, int32_t task,
                          int32_t n_folds, const void* configs, int32_t n_configs, uint64_t seed,
                          int32_t n_classes, int32_t trace_steps, int32_t n_threads, double* out_scores,
                          double* fold_scores, double* loss_trace, int32_t solver, int32_t metric) {
  const int32_t n_fits = n_configs * n_folds;
  std::vector<int32_t> fc((size_t)n_fits), ff((size_t)n_fits);
  for (int32_t i = 0; i < n_fits; ++i) { fc[i] = i / n_folds; ff[i] = i % n_folds; }
  std::vector<double> fs((size_t)n_fits);
  int rc = oracle_mlp_cv_fits_ex(mode, X, y, n, d, task, n_folds, configs, n_configs, seed, n_classes, fc.data(),
                                 ff.data(), n_fits, trace_steps, n_threads, fs.data(), loss_trace, nullptr, solver,
                                 metric);
  if (rc != 0) return rc;
  for (int32_t c = 0; c < n_configs; ++c) {
    if (mode == 1) {
      double a = 0.0;
      for (int32_t f = 0; f < n_folds; ++f) a = a + fs[(size_t)c * n_folds + f];
      out_scores[c] = a / (double)n_folds;
    } else {
      float a = 0.f;
      for (int32_t f = 0; f < n_folds; ++f) a = a + (float)fs[(size_t)c * n_folds + f];
      out_scores[c] = (double)(a / (float)n_folds);
    }
  }
  if (fold_scores) std::copy(fs.begin(), fs.end(), fold_scores);
  return 0;
}

int oracle_mlp_cv_eval(int32_t mode, const float* X, const float* y, int64_t n, int32_t d, int32_t task,
                       int32_t n_folds, const void* configs, int32_t n_configs, uint64_t seed,
                       int32_t n_classes, int32_t trace_steps, int32_t n_threads, double* out_scores,
                       double* fold_scores, double* loss_trace) {
  return oracle_mlp_cv_eval_ex(mode, X, y, n, d, task, n_folds, configs, n_configs, seed, n_classes, trace_steps,
                               n_threads, out_scores, fold_scores, loss_trace, 0, 0);
}

// Hold-out evaluation (paper sec. 6.2): one fit per configuration, trained on all n rows and scored
// on the n_test rows of (Xtest, ytest).  The random streams of these fits use the fold index
// HOLDOUT_FOLD_KEY, which no cross-validation fold can have.  theta_out: parameters of the last
// configuration's fit (or null).
enum : uint32_t { HOLDOUT_FOLD_KEY = 0xFFFFu };
int oracle_mlp_holdout_eval(int32_t mode, const float* X, const float* y, int64_t n, const float* Xtest,
                            const float* ytest, int64_t n_test, int32_t d, int32_t task, const void* configs,
                            int32_t n_configs, uint64_t seed, int32_t n_classes, int32_t solver, int32_t metric,
                            int32_t n_threads, double* out_scores, double* theta_out) {
  const Config* cfg = (const Config*)configs;
  if (!Xtest || !ytest || n_test < 1 || validate(X, y, n, d, task, 2, cfg, n_configs) != 0) return -1;
  if (solver < 0 || solver > 1 || metric < 0 || metric > 1) return -1;
  int32_t C = derive_classes(y, n, task, n_classes);
  if (C < 1) return -1;
  if (task == 0 && n_classes == 0) {  // labels of the test rows may exceed those seen in training
    const int32_t Ct = derive_classes(ytest, n_test, task, 0);
    if (Ct < 1) return -1;
    if (Ct > C) C = Ct;
  }
  std::vector<int32_t> pi;
  rng_perm((int32_t)n, seed, STREAM_FOLD, 0, 0, 0, pi);
#ifdef _OPENMP
  if (n_threads <= 0) n_threads = omp_get_num_procs();
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads)
#endif
  for (int32_t c = 0; c < n_configs; ++c) {
    double* tho = (theta_out && c == n_configs - 1) ? theta_out : nullptr;
    out_scores[c] = mode == 1
        ? run_fit<double>(X, y, n, d, C, task, 1, cfg[c], c, HOLDOUT_FOLD_KEY, seed, pi, 0, nullptr, tho, solver, metric, Xtest, ytest, n_test)
        : run_fit<float>(X, y, n, d, C, task, 1, cfg[c], c, HOLDOUT_FOLD_KEY, seed, pi, 0, nullptr, tho, solver, metric, Xtest, ytest, n_test);
  }
  return 0;
}

// Epoch order of a hold-out fit: the epoch permutation applied to the whole fold permutation.
int oracle_holdout_order(int64_t n, uint64_t seed, int32_t config, int32_t epoch, int32_t* out) {
  if (n < 1) return -1;
  std::vector<int32_t> pi, sigma;
  rng_perm((int32_t)n, seed, STREAM_FOLD, 0, 0, 0, pi);
  rng_perm((int32_t)n, seed, STREAM_PERM, (uint32_t)config, HOLDOUT_FOLD_KEY, (uint32_t)epoch, sigma);
  for (int64_t i = 0; i < n; ++i) out[i] = pi[sigma[(size_t)i]];
  return 0;
}

// n_steps momentum-SGD updates on P parameters with caller-supplied gradients grads[n_steps][P].
void oracle_sgd_steps(int32_t mode, int64_t P, int32_t n_steps, double lr, double momentum, double* theta,
                      double* vel, const double* grads) {
  if (mode == 1) {
    Sgd<double> a{lr, momentum};
    for (int32_t s = 0; s < n_steps; ++s) a.update(P, theta, vel, grads + (int64_t)s * P);
    return;
  }
  std::vector<float> th(theta, theta + P), vv(vel, vel + P), g((size_t)P);
  Sgd<float> a{(float)lr, (float)momentum};
  for (int32_t s = 0; s < n_steps; ++s) {
    for (int64_t i = 0; i < P; ++i) g[i] = (float)grads[(int64_t)s * P + i];
    a.update(P, th.data(), vv.data(), g.data());
  }
  for (int64_t i = 0; i < P; ++i) { theta[i] = th[i]; vel[i] = vv[i]; }
}

float oracle_tf32_round(float x) { return tf32_round(x); }
void oracle_tf32_split(float x, float* hi, float* lo) { tf32_split(x, hi, lo); }

int oracle_num_procs(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

}  // extern "C"
