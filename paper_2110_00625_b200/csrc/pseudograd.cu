// Learner level of Algorithm 1 with the stochastic gradient replaced by seeded variates:
//   w^j <- w^j - gamma g(seed, n, j, k, i),  k = 1..K,
// g an Irwin-Hall(4) variate of standard deviation sigma built from one SplitMix64 stream value
// (see mavg.h).  The K steps are applied in order to a value held in registers, so one pass over
// the replicas (8 bytes per element and learner) serves the whole round; the per-step rounding is
// the same as K separate passes.  The first pass after a (re-)broadcast reads w~ in place of
// every w^j ("set w^j = w~"), so the P copies need not exist before it.
#include "common.cuh"

namespace mavg {
namespace {

// (sum of the four 16-bit lanes of h - 131070) * c.  The lane sums are two 2-way 16-bit dot
// products with the weights (1, 1), chained through their addend, which starts at -131070
// (modular arithmetic: the same integer as extracting and adding the lanes one by one).
__device__ __forceinline__ float ih4(uint64_t h, float c) {
  const uint32_t lo = (uint32_t)h, hi = (uint32_t)(h >> 32);
  const uint32_t s = __dp2a_lo(hi, 0x0101u, __dp2a_lo(lo, 0x0101u, (uint32_t)-131070));
  return (float)(int32_t)s * c;
}

// grid = (x, P); dynamic shared memory holds the K step keys of learner blockIdx.y.
// MOM: learner-level momentum, u^j read (unless mom.read_u == 0) and written once per pass like w^j.
template <bool MOM>
__global__ void __launch_bounds__(256)
k_pseudograd_steps(float* rep, int64_t stride, const float* src, int64_t src_stride, int64_t n,
                   int K, uint64_t seed, int64_t round, int k_first, float c, float gamma,
                   const MomArgs mom) {
  extern __shared__ uint64_t keys[];
  const int j = blockIdx.y;
  const uint64_t lk = learner_key(seed, kTagPseudoGrad, (uint64_t)round, (uint64_t)j);
  for (int k = threadIdx.x; k < K; k += blockDim.x) keys[k] = fold(lk, (uint64_t)(k_first + k));
  __syncthreads();
  float* row = rep + (size_t)j * stride;
  float4* row4 = reinterpret_cast<float4*>(row);
  const float* in = src + (size_t)j * src_stride;
  const float4* in4 = reinterpret_cast<const float4*>(in);
  const int64_t n4 = n >> 2;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  const float ng = -gamma;
  float* urow = MOM ? mom.u + (size_t)j * mom.u_stride : nullptr;
  float4* urow4 = reinterpret_cast<float4*>(urow);
  for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += step) {
    float4 w = src_stride ? __ldcs(in4 + q) : __ldg(in4 + q);
    float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
    if (MOM && mom.read_u) u = __ldcs(urow4 + q);
    const uint64_t c0 = (uint64_t)(4 * q + 1) * kGamma;  // element i uses (i+1) G
    for (int k = 0; k < K; ++k) {
      const uint64_t key = keys[k];
      const float g0 = ih4(mix64(key + c0), c), g1 = ih4(mix64(key + c0 + kGamma), c);
      const float g2 = ih4(mix64(key + c0 + 2 * kGamma), c);
      const float g3 = ih4(mix64(key + c0 + 3 * kGamma), c);
      if (MOM) {
        msgd(w.x, u.x, g0, gamma, mom.beta);
        msgd(w.y, u.y, g1, gamma, mom.beta);
        msgd(w.z, u.z, g2, gamma, mom.beta);
        msgd(w.w, u.w, g3, gamma, mom.beta);
      } else {
        w.x = fmaf(ng, g0, w.x);
        w.y = fmaf(ng, g1, w.y);
        w.z = fmaf(ng, g2, w.z);
        w.w = fmaf(ng, g3, w.w);
      }
    }
    __stcs(row4 + q, w);
    if (MOM) __stcs(urow4 + q, u);
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {
    const int64_t i = (n4 << 2) + threadIdx.x;
    float w = in[i];
    float u = (MOM && mom.read_u) ? urow[i] : 0.f;
    for (int k = 0; k < K; ++k) {
      const float gk = ih4(fold(keys[k], (uint64_t)i), c);
      if (MOM) msgd(w, u, gk, gamma, mom.beta);
      else w = fmaf(ng, gk, w);
    }
    row[i] = w;
    if (MOM) urow[i] = u;
  }
}

}  // namespace

cudaError_t launch_pseudograd_steps(mavg_ctx* c, int64_t round) {
  const int64_t n = c->cfg.n;
  const int P = c->cfg.P, K = c->cfg.K;
  const double var_lane = (65536.0 * 65536.0 - 1.0) / 12.0;
  const float scale = (float)((double)c->cfg.pseudo_grad_sigma / sqrt(4.0 * var_lane));
  constexpr int kMaxFused = 2048;  // step keys per launch (16 KB of shared memory)
  int64_t blocks_x = ((n >> 2) + 255) / 256;
  int64_t cap = ((int64_t)c->sm_count * 8 + P - 1) / P;
  if (blocks_x > cap) blocks_x = cap;
  if (blocks_x < 1) blocks_x = 1;
  for (int k0 = 0; k0 < K; k0 += kMaxFused) {
    int kc = K - k0 < kMaxFused ? K - k0 : kMaxFused;
    dim3 grid((unsigned)blocks_x, (unsigned)P);
    const bool from_global = c->replicas_equal_global;
    const MomArgs mom = mom_args(c, from_global);
    prof_begin(c, MAVG_K_PSEUDOGRAD);
    if (mom.u)
      k_pseudograd_steps<true><<<grid, 256, (size_t)kc * sizeof(uint64_t), c->stream>>>(
          c->buf.replicas, c->buf.replica_stride, from_global ? c->buf.global_w : c->buf.replicas,
          from_global ? 0 : c->buf.replica_stride, n, kc, c->cfg.seed, round, k0 + 1, scale,
          c->cfg.local_lr, mom);
    else
      k_pseudograd_steps<false><<<grid, 256, (size_t)kc * sizeof(uint64_t), c->stream>>>(
          c->buf.replicas, c->buf.replica_stride, from_global ? c->buf.global_w : c->buf.replicas,
          from_global ? 0 : c->buf.replica_stride, n, kc, c->cfg.seed, round, k0 + 1, scale,
          c->cfg.local_lr, mom);
    prof_end(c);
    c->replicas_equal_global = false;
    c->replicas_materialized = true;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace mavg
