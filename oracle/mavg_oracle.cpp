// M-AVG oracle: a plain, slow CPU statement of Algorithm 1 (K-step averaging SGD with block
// momentum) and of the synthetic objectives it is exercised on.
//
// THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library has something independent to
// be compared with.  It shares no code, header, table or constant generator with the CUDA path,
// and only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
//
// Conventions (the paper's notation):
//   P learners (j = 0..P-1 here, 1..P in the paper), K local steps (k = 1..K), minibatch B
//   (s = 0..B-1), round n = 1..N, local step size gamma, block momentum mu; w~ is the global
//   model, v the block-momentum buffer, w^j the replica of learner j.  The block learning rate
//   zeta is an extension (zeta = 1 is exactly Algorithm 1): v <- mu v + zeta d.
//
// Arithmetic: all state (w~, v, replicas, activations) is stored in fp32; every dot product, row
// sum and sum over learners is accumulated in double and rounded to fp32 once when stored.
// Nothing here is blocked, fused or reordered beyond what the algorithm states.
//
// Parity status of each function is listed in the header of oracle.py next to the pin that
// covers it; the free-running MLP trajectories are "parity unpinned" (the paper prints no loss
// or weight value for any workload).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// Counter-based random numbers: SplitMix64 (Steele, Lea, Flood, OOPSLA 2014).  The generator's
// i-th output from state s0 is mix64(s0 + i*GAMMA), i = 1, 2, ...; that makes it addressable by
// counter.  A stream key is obtained by folding the counters (tag, round, learner, step) into the
// seed, each fold being one generator step: fold(s, c) = mix64(s + (c+1)*GAMMA).
// ---------------------------------------------------------------------------------------------
constexpr uint64_t GAMMA = 0x9E3779B97F4A7C15ull;

inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
inline uint64_t fold(uint64_t s, uint64_t c) { return mix64(s + (c + 1) * GAMMA); }

constexpr uint64_t TAG_BATCH = 1;       // minibatch sample indices
constexpr uint64_t TAG_PSEUDOGRAD = 2;  // synthetic stochastic gradients

inline uint64_t stream_key(uint64_t seed, uint64_t tag, uint64_t n, uint64_t j, uint64_t k) {
  return fold(fold(fold(fold(seed, tag), n), j), k);
}

// Learner j owns the contiguous sample range [floor(j S / P), floor((j+1) S / P)).
inline void shard(int64_t S, int32_t P, int32_t j, int64_t* lo, int64_t* hi) {
  *lo = (int64_t)(((__int128)j * S) / P);
  *hi = (int64_t)(((__int128)(j + 1) * S) / P);
}

// "randomly sample a mini-batch of size B_n" (Algorithm 1): i.i.d. uniform with replacement in
// the learner's shard.  u = top 32 bits of the stream value; idx = lo + floor(u * len / 2^32).
inline int32_t batch_index(uint64_t key, int32_t s, int64_t lo, int64_t len) {
  uint64_t u = fold(key, (uint64_t)s) >> 32;
  return (int32_t)(lo + (int64_t)((u * (uint64_t)len) >> 32));
}

// Irwin-Hall(4) variate scaled to standard deviation sigma: the sum of the four 16-bit lanes of
// one 64-bit stream value, centred, times one fp32 constant.  Integer arithmetic followed by a
// single fp32 multiply, so every IEEE machine gets the same bits.
inline float ih4_scale(float sigma) {
  const double var_lane = (65536.0 * 65536.0 - 1.0) / 12.0;  // variance of uniform{0..65535}
  return (float)((double)sigma / std::sqrt(4.0 * var_lane));
}
inline float ih4(uint64_t h, float c) {
  int32_t S = (int32_t)(h & 0xFFFF) + (int32_t)((h >> 16) & 0xFFFF) +
              (int32_t)((h >> 32) & 0xFFFF) + (int32_t)(h >> 48);
  return (float)(S - 131070) * c;
}

// Round-to-nearest-even fp32 -> bf16 -> fp32 (NaN kept quiet).
inline float bf16r(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) {
    u |= 0x00400000u;
    u &= 0xFFFF0000u;
  } else {
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
  }
  float y;
  std::memcpy(&y, &u, 4);
  return y;
}

// ---------------------------------------------------------------------------------------------
// Objective: an MLP with bias, ReLU between layers, softmax cross-entropy averaged over the
// minibatch (the 1/B_n of Algorithm 1's update).  Flat parameter layout per replica:
// [W_1 (out x in, row-major), b_1, W_2, b_2, ...].
// ---------------------------------------------------------------------------------------------
int64_t mlp_param_count(int L, const int32_t* dims) {
  int64_t n = 0;
  for (int l = 0; l < L; ++l) n += (int64_t)dims[l + 1] * dims[l] + dims[l + 1];
  return n;
}

// Minibatch-mean gradient and loss at w.  X is the gathered minibatch [B, dims[0]], y its labels.
// bf16 != 0: every operand of a matrix product is rounded to bf16 first (weights, activations,
// dZ); products are exact and accumulate in double; bias, ReLU, softmax and the bias gradient
// stay in fp32/double.
void mlp_loss_grad(int L, const int32_t* dims, const float* w, const float* X, const int32_t* y,
                   int B, int bf16, float* grad, double* loss_out) {
  auto q = [bf16](float x) { return bf16 ? bf16r(x) : x; };
  std::vector<const float*> W(L), bias(L);
  std::vector<int64_t> offW(L), offb(L);
  {
    int64_t off = 0;
    for (int l = 0; l < L; ++l) {
      offW[l] = off;
      W[l] = w + off;
      off += (int64_t)dims[l + 1] * dims[l];
      offb[l] = off;
      bias[l] = w + off;
      off += dims[l + 1];
    }
  }
  // act[l] = A_l as the next matrix product sees it (rounded in bf16 mode); z[l] = Z_l in fp32.
  std::vector<std::vector<float>> act(L + 1), z(L + 1);
  act[0].resize((size_t)B * dims[0]);
  for (size_t i = 0; i < act[0].size(); ++i) act[0][i] = q(X[i]);
  for (int l = 1; l <= L; ++l) {
    const int in = dims[l - 1], out = dims[l];
    z[l].resize((size_t)B * out);
    act[l].resize((size_t)B * out);
    for (int b = 0; b < B; ++b)
      for (int o = 0; o < out; ++o) {
        double acc = 0.0;
        const float* wr = W[l - 1] + (size_t)o * in;
        const float* ar = act[l - 1].data() + (size_t)b * in;
        for (int i = 0; i < in; ++i) acc += (double)q(wr[i]) * (double)ar[i];
        float zz = (float)(acc + (double)bias[l - 1][o]);
        z[l][(size_t)b * out + o] = zz;
        act[l][(size_t)b * out + o] = (l < L) ? q(zz > 0.f ? zz : 0.f) : zz;
      }
  }
  // softmax cross-entropy, log-sum-exp with the maximum subtracted; dZ_L = (p - onehot) / B
  const int C = dims[L];
  std::vector<float> dz((size_t)B * C);
  double loss = 0.0;
  for (int b = 0; b < B; ++b) {
    const float* lg = z[L].data() + (size_t)b * C;
    double m = lg[0];
    for (int c = 1; c < C; ++c) m = lg[c] > m ? lg[c] : m;
    double se = 0.0;
    for (int c = 0; c < C; ++c) se += std::exp((double)lg[c] - m);
    double lse = m + std::log(se);
    loss += lse - (double)lg[y[b]];
    for (int c = 0; c < C; ++c) {
      double p = std::exp((double)lg[c] - lse);
      dz[(size_t)b * C + c] = (float)((p - (c == y[b] ? 1.0 : 0.0)) / (double)B);
    }
  }
  *loss_out = loss / (double)B;
  // backward, layer L down to 1
  for (int l = L; l >= 1; --l) {
    const int in = dims[l - 1], out = dims[l];
    float* gW = grad + offW[l - 1];
    float* gb = grad + offb[l - 1];
    for (int o = 0; o < out; ++o) {
      double acc = 0.0;
      for (int b = 0; b < B; ++b) acc += (double)dz[(size_t)b * out + o];
      gb[o] = (float)acc;
    }
    for (int o = 0; o < out; ++o)
      for (int i = 0; i < in; ++i) {
        double acc = 0.0;
        for (int b = 0; b < B; ++b)
          acc += (double)q(dz[(size_t)b * out + o]) * (double)act[l - 1][(size_t)b * in + i];
        gW[(size_t)o * in + i] = (float)acc;
      }
    if (l > 1) {
      std::vector<float> dzp((size_t)B * in);
      for (int b = 0; b < B; ++b)
        for (int i = 0; i < in; ++i) {
          double acc = 0.0;
          for (int o = 0; o < out; ++o)
            acc += (double)q(dz[(size_t)b * out + o]) * (double)q(W[l - 1][(size_t)o * in + i]);
          // ReLU'(0) = 0
          dzp[(size_t)b * in + i] = z[l - 1][(size_t)b * in + i] > 0.f ? (float)acc : 0.f;
        }
      dz.swap(dzp);
    }
  }
}

inline void sgd_step(float* w, const float* g, int64_t n, float gamma) {
  for (int64_t i = 0; i < n; ++i) w[i] = (float)((double)w[i] - (double)gamma * (double)g[i]);
}

// Learner-level momentum (the variant named after Eq. 2 and in the conclusion: momentum SGD in
// place of plain SGD inside each learner), written in the form Eq. 2 uses at the meta level:
//   u <- beta u - gamma g;  w <- w + u.
inline void msgd_step(float* w, float* u, const float* g, int64_t n, float gamma, float beta) {
  for (int64_t i = 0; i < n; ++i) {
    const float un = (float)((double)beta * (double)u[i] - (double)gamma * (double)g[i]);
    u[i] = un;
    w[i] = (float)((double)w[i] + (double)un);
  }
}

}  // namespace

extern "C" {

enum { ORC_OBJ_PSEUDOGRAD = 1, ORC_OBJ_MLP = 2, ORC_OBJ_QUADRATIC = 3 };

// One M-AVG problem.  Pointers are host memory owned by the caller.
struct orc_problem {
  int32_t P, K, B;
  float gamma, zeta, mu;
  uint64_t seed;
  int32_t objective;
  int64_t n;        // parameters per replica
  int64_t stride;   // floats between consecutive replicas (>= n)
  // MLP
  int32_t n_layers;
  int32_t dims[9];
  int32_t bf16;
  const float* x;   // [S, dims[0]]
  const int32_t* y; // [S]
  int64_t S;
  // pseudo-gradient
  float sigma;
  // quadratic F(w) = 1/2 sum_i a_i w_i^2, exact gradient (used only to pin the round loop)
  const float* quad_a;
  int32_t threads;  // OpenMP threads over the independent learners (<= 0: library default)
  // learner-level momentum (0 = plain SGD, Algorithm 1 as printed)
  float beta;
  int32_t reset_u;  // 1: u^j <- 0 at the start of every round; 0: u^j carried over the rounds
  float* u;         // [P, stride] learner momentum buffers; required when beta != 0
};

uint64_t orc_mix64(uint64_t z) { return mix64(z); }
uint64_t orc_splitmix64_output(uint64_t state0, uint64_t i) { return mix64(state0 + i * GAMMA); }
uint64_t orc_stream_key(uint64_t seed, uint64_t tag, uint64_t n, uint64_t j, uint64_t k) {
  return stream_key(seed, tag, n, j, k);
}
float orc_bf16_round(float x) { return bf16r(x); }
void orc_bf16_round_array(const float* in, float* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16r(in[i]);
}
void orc_shard_bounds(int64_t S, int32_t P, int32_t j, int64_t* lo, int64_t* hi) {
  shard(S, P, j, lo, hi);
}
// The B sample indices learner j draws at local step k (1-based) of round n (1-based).
void orc_batch_indices(uint64_t seed, int64_t n, int32_t P, int32_t j, int32_t k, int64_t S,
                       int32_t B, int32_t* out) {
  int64_t lo, hi;
  shard(S, P, j, &lo, &hi);
  uint64_t key = stream_key(seed, TAG_BATCH, (uint64_t)n, (uint64_t)j, (uint64_t)k);
  for (int32_t s = 0; s < B; ++s) out[s] = batch_index(key, s, lo, hi - lo);
}
// Elements [i0, i0+count) of learner j's synthetic gradient at step k of round n.
void orc_pseudograd(uint64_t seed, int64_t n, int32_t j, int32_t k, int64_t i0, int64_t count,
                    float sigma, float* out) {
  uint64_t key = stream_key(seed, TAG_PSEUDOGRAD, (uint64_t)n, (uint64_t)j, (uint64_t)k);
  float c = ih4_scale(sigma);
  for (int64_t i = 0; i < count; ++i) out[i] = ih4(fold(key, (uint64_t)(i0 + i)), c);
}
int64_t orc_mlp_param_count(int32_t L, const int32_t* dims) { return mlp_param_count(L, dims); }
void orc_mlp_loss_grad(int32_t L, const int32_t* dims, const float* w, const float* X,
                       const int32_t* y, int32_t B, int32_t bf16, float* grad, double* loss) {
  mlp_loss_grad(L, dims, w, X, y, B, bf16, grad, loss);
}

// Learner level of Algorithm 1: every learner, independently, takes K minibatch-SGD steps on its
// own replica:  w^j <- w^j - gamma * (1/B) sum_s grad F(w^j; xi^j_{k,s}),  k = 1..K.
// losses[j*K + (k-1)] receives the minibatch loss seen at step k (MLP only, else 0).
// G (n doubles, may be null) receives G_n of Eq. 2: (1/(B P)) sum_j sum_k sum_s grad F, i.e. the
// mean over learners of the summed minibatch-mean gradients, accumulated apart from the weights.
void orc_local_steps(const orc_problem* pb, int64_t round, float* replicas, double* losses,
                     double* G) {
  const int P = pb->P, K = pb->K;
  const int64_t n = pb->n;
  std::vector<std::vector<double>> Gj;
  if (G) Gj.assign(P, std::vector<double>((size_t)n, 0.0));
#ifdef _OPENMP
  int nt = pb->threads > 0 ? pb->threads : omp_get_max_threads();
  if (nt > P) nt = P;
#pragma omp parallel for num_threads(nt) schedule(static)
#endif
  for (int j = 0; j < P; ++j) {
    float* w = replicas + (size_t)j * pb->stride;
    float* u = pb->beta != 0.f ? pb->u + (size_t)j * pb->stride : nullptr;
    if (u && pb->reset_u)
      for (int64_t i = 0; i < n; ++i) u[i] = 0.f;
    std::vector<float> g((size_t)n);
    std::vector<float> X;
    std::vector<int32_t> idx, yb;
    for (int k = 1; k <= K; ++k) {
      double loss = 0.0;
      if (pb->objective == ORC_OBJ_MLP) {
        const int d0 = pb->dims[0];
        idx.resize(pb->B);
        yb.resize(pb->B);
        X.resize((size_t)pb->B * d0);
        orc_batch_indices(pb->seed, round, P, j, k, pb->S, pb->B, idx.data());
        for (int s = 0; s < pb->B; ++s) {
          std::memcpy(&X[(size_t)s * d0], pb->x + (size_t)idx[s] * d0, sizeof(float) * d0);
          yb[s] = pb->y[idx[s]];
        }
        mlp_loss_grad(pb->n_layers, pb->dims, w, X.data(), yb.data(), pb->B, pb->bf16, g.data(),
                      &loss);
      } else if (pb->objective == ORC_OBJ_PSEUDOGRAD) {
        orc_pseudograd(pb->seed, round, j, k, 0, n, pb->sigma, g.data());
      } else {  // ORC_OBJ_QUADRATIC
        for (int64_t i = 0; i < n; ++i) g[i] = (float)((double)pb->quad_a[i] * (double)w[i]);
      }
      if (G)
        for (int64_t i = 0; i < n; ++i) Gj[j][i] += (double)g[i];
      if (u)
        msgd_step(w, u, g.data(), n, pb->gamma, pb->beta);
      else
        sgd_step(w, g.data(), n, pb->gamma);
      if (losses) losses[(size_t)j * K + (k - 1)] = loss;
    }
  }
  if (G)
    for (int64_t i = 0; i < n; ++i) {
      double acc = 0.0;
      for (int j = 0; j < P; ++j) acc += Gj[j][i];
      G[i] = acc / (double)P;
    }
}

// Meta level of Algorithm 1, followed by the next round's "set w^j = w~":
//   a = (1/P) sum_j w^j;  d = a - w~;  v <- mu v + zeta d;  w~ <- w~ + v;  w^j <- w~.
// d is evaluated as (sum_j (w^j - w~)) / P, the same real number, in double.
void orc_meta_update(int32_t P, int64_t n, int64_t stride, float* replicas, float* w, float* v,
                     float mu, float zeta) {
  for (int64_t i = 0; i < n; ++i) {
    double acc = 0.0;
    for (int j = 0; j < P; ++j) acc += (double)replicas[(size_t)j * stride + i] - (double)w[i];
    double d = acc / (double)P;
    float vn = (float)((double)mu * (double)v[i] + (double)zeta * d);
    float wn = (float)((double)w[i] + (double)vn);
    v[i] = vn;
    w[i] = wn;
    for (int j = 0; j < P; ++j) replicas[(size_t)j * stride + i] = wn;
  }
}

// Algorithm 1's initialisation: v <- 0 and every replica set to w~_1.
void orc_init(int32_t P, int64_t n, int64_t stride, float* replicas, const float* w, float* v) {
  for (int64_t i = 0; i < n; ++i) v[i] = 0.f;
  for (int j = 0; j < P; ++j) std::memcpy(replicas + (size_t)j * stride, w, sizeof(float) * n);
}

// One round n of Algorithm 1.  mean_loss = mean over the P*K minibatch losses of the round.
void orc_round(const orc_problem* pb, int64_t round, float* replicas, float* w, float* v,
               double* mean_loss, double* G) {
  std::vector<double> losses((size_t)pb->P * pb->K, 0.0);
  orc_local_steps(pb, round, replicas, losses.data(), G);
  double acc = 0.0;
  for (double l : losses) acc += l;
  if (mean_loss) *mean_loss = acc / (double)losses.size();
  orc_meta_update(pb->P, pb->n, pb->stride, replicas, w, v, pb->mu, pb->zeta);
}

int32_t orc_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
