// Meta level of Algorithm 1 fused with the next round's "set w^j = w~":
//   a = (1/P) sum_j w^j;  d = a - w~;  v <- mu v + zeta d;  w~ <- w~ + v;  w^j <- w~  for all j.
// One pass over HBM: per element 4P + 8 bytes read (4P + 4 when mu = 0: v is not read) and
// 4P + 8 bytes written.  d is formed as (sum_j (w^j - w~)) / P in ascending j, which is the same
// real number and keeps the fp32 sum small.
#include "common.cuh"

namespace mavg {
namespace {

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

__device__ __forceinline__ float4 sub4(float4 a, float4 b) {
  return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
}
__device__ __forceinline__ void acc4(float4& a, float4 b) {
  a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
}

__device__ __forceinline__ void meta_scalar(float* rep, int64_t stride, float* w, float* v, int P,
                                            int64_t i, float mu, float zeta, float inv_p,
                                            bool read_v) {
  float wt = w[i], acc = 0.f;
  for (int j = 0; j < P; ++j) acc += rep[(size_t)j * stride + i] - wt;
  float d = acc * inv_p;
  float vn = read_v ? fmaf(mu, v[i], zeta * d) : zeta * d;
  float wn = wt + vn;
  v[i] = vn;
  w[i] = wn;
  for (int j = 0; j < P; ++j) rep[(size_t)j * stride + i] = wn;
}

// U replica loads are kept in flight per thread; STREAM_ST selects evict-first stores for the
// broadcast (replica sets far larger than L2) or plain stores (sets the next kernel re-reads).
template <int U, bool STREAM_ST>
__global__ void __launch_bounds__(256)
k_meta_update(float* __restrict__ rep, int64_t stride, float* __restrict__ w,
              float* __restrict__ v, int P, int64_t n, float mu, float zeta, float inv_p,
              int read_v) {
  const int64_t n4 = n >> 2;
  const int64_t stride4 = stride >> 2;
  float4* rep4 = reinterpret_cast<float4*>(rep);
  float4* w4 = reinterpret_cast<float4*>(w);
  float4* v4 = reinterpret_cast<float4*>(v);
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += step) {
    const float4 wt = ld_stream(w4 + q);
    float4 vt = make_float4(0.f, 0.f, 0.f, 0.f);
    if (read_v) vt = ld_stream(v4 + q);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4* rq = rep4 + q;
    int j0 = 0;
    for (; j0 + U <= P; j0 += U) {
      float4 r[U];
#pragma unroll
      for (int u = 0; u < U; ++u) r[u] = ld_stream(rq + (size_t)(j0 + u) * stride4);
#pragma unroll
      for (int u = 0; u < U; ++u) acc4(acc, sub4(r[u], wt));
    }
    for (; j0 < P; ++j0) acc4(acc, sub4(ld_stream(rq + (size_t)j0 * stride4), wt));
    float4 vn, wn;
    vn.x = fmaf(mu, vt.x, zeta * (acc.x * inv_p));
    vn.y = fmaf(mu, vt.y, zeta * (acc.y * inv_p));
    vn.z = fmaf(mu, vt.z, zeta * (acc.z * inv_p));
    vn.w = fmaf(mu, vt.w, zeta * (acc.w * inv_p));
    wn.x = wt.x + vn.x; wn.y = wt.y + vn.y; wn.z = wt.z + vn.z; wn.w = wt.w + vn.w;
    if (STREAM_ST) {
      __stcs(v4 + q, vn);
      __stcs(w4 + q, wn);
      for (int j = 0; j < P; ++j) __stcs(rep4 + (size_t)j * stride4 + q, wn);
    } else {
      v4[q] = vn;
      w4[q] = wn;
      for (int j = 0; j < P; ++j) rep4[(size_t)j * stride4 + q] = wn;
    }
  }
  // ragged tail (n not a multiple of 4)
  if (blockIdx.x == 0 && threadIdx.x < (n & 3))
    meta_scalar(rep, stride, w, v, P, (n4 << 2) + threadIdx.x, mu, zeta, inv_p, read_v != 0);
}

// Algorithm 1's "set w^j = w~" on its own (initialisation, resume), optionally with v <- 0.
__global__ void __launch_bounds__(256)
k_broadcast(float* __restrict__ rep, int64_t stride, const float* __restrict__ w,
            float* __restrict__ v, int P, int64_t n, int zero_v) {
  const int64_t n4 = n >> 2;
  const int64_t stride4 = stride >> 2;
  float4* rep4 = reinterpret_cast<float4*>(rep);
  const float4* w4 = reinterpret_cast<const float4*>(w);
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += step) {
    float4 wt = w4[q];
    if (zero_v) reinterpret_cast<float4*>(v)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < P; ++j) rep4[(size_t)j * stride4 + q] = wt;
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {
    int64_t i = (n4 << 2) + threadIdx.x;
    if (zero_v) v[i] = 0.f;
    for (int j = 0; j < P; ++j) rep[(size_t)j * stride + i] = w[i];
  }
}

int grid_for(const mavg_ctx* c, int64_t work_items, int threads, int blocks_per_sm) {
  int64_t need = (work_items + threads - 1) / threads;
  int64_t cap = (int64_t)c->sm_count * blocks_per_sm;
  if (need < 1) need = 1;
  return (int)(need < cap ? need : cap);
}

}  // namespace

cudaError_t launch_broadcast(mavg_ctx* c, bool zero_v) {
  const int64_t n = c->cfg.n;
  int grid = grid_for(c, n >> 2, 256, 8);
  prof_begin(c, MAVG_K_BROADCAST);
  k_broadcast<<<grid, 256, 0, c->stream>>>(c->buf.replicas, c->buf.replica_stride,
                                           c->buf.global_w, c->buf.momentum, c->cfg.P, n,
                                           zero_v ? 1 : 0);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_meta_update(mavg_ctx* c) {
  const int64_t n = c->cfg.n;
  const int P = c->cfg.P;
  const float mu = c->cfg.mu, zeta = c->cfg.block_lr;
  const float inv_p = 1.0f / (float)P;
  const int read_v = mu != 0.f ? 1 : 0;
  int grid = grid_for(c, n >> 2, 256, 6);
  // A replica set that fits in L2 is about to be re-read by the next round's first local step:
  // keep it there.  Larger sets are written with evict-first stores.
  const bool stream_st = (size_t)P * (size_t)n * 4 > c->l2_bytes / 2;
  prof_begin(c, MAVG_K_META);
  if (stream_st)
    k_meta_update<8, true><<<grid, 256, 0, c->stream>>>(c->buf.replicas, c->buf.replica_stride,
                                                        c->buf.global_w, c->buf.momentum, P, n,
                                                        mu, zeta, inv_p, read_v);
  else
    k_meta_update<8, false><<<grid, 256, 0, c->stream>>>(c->buf.replicas, c->buf.replica_stride,
                                                         c->buf.global_w, c->buf.momentum, P, n,
                                                         mu, zeta, inv_p, read_v);
  prof_end(c);
  return cudaGetLastError();
}

}  // namespace mavg
