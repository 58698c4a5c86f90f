// Meta level of Algorithm 1 fused with the next round's "set w^j = w~":
//   a = (1/P) sum_j w^j;  d = a - w~;  v <- mu v + zeta d;  w~ <- w~ + v;  w^j <- w~  for all j.
// One pass over HBM: per element 4P + 8 bytes read (4P + 4 when mu = 0: v is not read) and
// 4P + 8 bytes written (8 when the P copies are left to the next round's first local step).  d is formed as (sum_j (w^j - w~)) / P in ascending j, which is the same
// real number and keeps the fp32 sum small.
#include "common.cuh"
#include "tc_ptx.cuh"

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
                                            bool read_v, bool bcast) {
  float wt = w[i], acc = 0.f;
  for (int j = 0; j < P; ++j) acc += rep[(size_t)j * stride + i] - wt;
  float d = acc * inv_p;
  float vn = read_v ? fmaf(mu, v[i], zeta * d) : zeta * d;
  float wn = wt + vn;
  v[i] = vn;
  w[i] = wn;
  if (bcast)
    for (int j = 0; j < P; ++j) rep[(size_t)j * stride + i] = wn;
}

// U replica loads are kept in flight per thread; STREAM_ST selects evict-first stores for the
// broadcast (replica sets far larger than L2) or plain stores (sets the next kernel re-reads).
// SHADOW: also writes the bf16 copy of the new w~'s weight matrices (see ShadowMap), which saves
// the separate pass that would read w~ again.
template <int U, bool STREAM_ST, bool SHADOW = false>
__global__ void __launch_bounds__(256)
k_meta_update(float* __restrict__ rep, int64_t stride, float* __restrict__ w,
              float* __restrict__ v, int P, int64_t n, float mu, float zeta, float inv_p,
              int read_v, int bcast, const ShadowMap sm = ShadowMap()) {
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
      if (bcast)
        for (int j = 0; j < P; ++j) __stcs(rep4 + (size_t)j * stride4 + q, wn);
    } else {
      v4[q] = vn;
      w4[q] = wn;
      if (bcast)
        for (int j = 0; j < P; ++j) rep4[(size_t)j * stride4 + q] = wn;
    }
    if (SHADOW) {
      const int64_t i = q << 2;
      for (int l = 0; l < sm.L; ++l) {
        const int64_t r = i - sm.w_off[l];
        if (r >= 0 && r < sm.total[l]) {
          __nv_bfloat162 h0 = __floats2bfloat162_rn(wn.x, wn.y), h1 = __floats2bfloat162_rn(wn.z, wn.w);
          *reinterpret_cast<uint2*>(sm.dst + sm.sh_off[l] + r) =
              make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
          break;
        }
      }
    }
  }
  // ragged tail (n not a multiple of 4)
  if (blockIdx.x == 0 && threadIdx.x < (n & 3))
    meta_scalar(rep, stride, w, v, P, (n4 << 2) + threadIdx.x, mu, zeta, inv_p, read_v != 0,
                bcast != 0);
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

// ---- the same update driven by bulk copies ------------------------------------------------------
// One block per SM walks over tiles of T consecutive elements.  A producer warp keeps a ring of
// STAGES shared-memory stages filled with G replica tiles each (cp.async.bulk, completion counted
// on mbarriers) plus the tile of w~ and v; THREADS consumer threads add the differences
// w^j - w~ in ascending j, form v and w~, and one thread sends the two result tiles back and
// the w~ tile to every replica with bulk stores.  Bytes in flight per SM are set by the ring
// (tens of KB), not by registers, which is what a pass with 2P+4 concurrent streams needs.
// What is left of n after the last whole tile is done by the consumers of the last block with
// plain loads and stores (the same arithmetic in the same order).
enum { ERR_META_PRODUCER = 31, ERR_META_CONSUMER = 32 };

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes,
                                          uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(tc::smem_u32(src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_plain(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc::smem_u32(bar)) : "memory");
}
// Barrier 1 over the `threads` consumer threads that also ORs a predicate over them: every
// consumer learns whether any of them gave up a wait, so that they all leave the tile loop in the
// same iteration and nobody is left behind at a counted barrier.
__device__ __forceinline__ bool consumers_any(bool pred, int threads) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
      "barrier.red.or.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(threads)
      : "memory");
  return r != 0;
}

template <int T, int G, int STAGES, int THREADS>
__global__ void __launch_bounds__(THREADS + 32)
k_meta_update_bulk(float* __restrict__ rep, int64_t stride, float* __restrict__ w,
                   float* __restrict__ v, int P, int64_t n, float mu, float zeta,
                   float inv_p, int read_v, int bcast, int* status) {
  extern __shared__ __align__(128) uint8_t sm[];
  float* st_rep = reinterpret_cast<float*>(sm);            // [STAGES][G][T]
  float* st_wv = st_rep + (size_t)STAGES * G * T;          // [2][2][T]: (w~, v) of two tiles
  float* st_out = st_wv + 4 * T;                           // [2][2][T]: (new w~, new v)
  __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], wv_full[2], wv_empty[2];
  __shared__ int abort_flag;
  constexpr int kWarps = THREADS / 32;
  constexpr int PER = T / THREADS;                          // elements per thread, multiple of 4
  const int tid = threadIdx.x;
  const int64_t n_tiles = n / T;
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      tc::mbar_init(&full[s], 1);
      tc::mbar_init(&empty[s], kWarps);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(&wv_full[b], 1);
      tc::mbar_init(&wv_empty[b], kWarps);
    }
    abort_flag = 0;
    tc::fence_barrier_init();
    tc::fence_proxy_async();
  }
  __syncthreads();
  volatile int* abortp = &abort_flag;
  const int groups = (P + G - 1) / G;
  if (tid >= THREADS) {                                     // producer warp
    if (tid == THREADS) {
      uint32_t sc = 0, tcount = 0;
      for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tcount) {
        const int b = tcount & 1;
        if (!tc::mbar_wait(&wv_empty[b], ((tcount >> 1) & 1) ^ 1, abortp, status, ERR_META_PRODUCER))
          return;
        tc::mbar_arrive_expect_tx(&wv_full[b], (read_v ? 2 : 1) * T * 4);
        bulk_load(st_wv + (size_t)(b * 2) * T, w + t * T, T * 4, &wv_full[b]);
        if (read_v) bulk_load(st_wv + (size_t)(b * 2 + 1) * T, v + t * T, T * 4, &wv_full[b]);
        for (int gi = 0; gi < groups; ++gi, ++sc) {
          const int s = sc % STAGES;
          if (!tc::mbar_wait(&empty[s], ((sc / STAGES) & 1) ^ 1, abortp, status, ERR_META_PRODUCER))
            return;
          const int cnt = min(G, P - gi * G);
          tc::mbar_arrive_expect_tx(&full[s], (uint32_t)cnt * T * 4);
          for (int u = 0; u < cnt; ++u)
            bulk_load(st_rep + ((size_t)s * G + u) * T, rep + (size_t)(gi * G + u) * stride + t * T,
                      T * 4, &full[s]);
        }
      }
    }
    return;
  }
  // Consumers.  A consumer whose wait is abandoned does not leave on its own: it carries `failed`
  // to the tile's first barrier, which tells every consumer, and they all leave together there
  // (before anything of the tile is stored).  The producer's waits end through abort_flag.
  uint32_t sc = 0, tcount = 0;
  const int lane = tid & 31;
  for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tcount) {
    const int b = tcount & 1;
    bool failed = !tc::mbar_wait(&wv_full[b], (tcount >> 1) & 1, abortp, status, ERR_META_CONSUMER);
    float wt[PER], acc[PER];
#pragma unroll
    for (int i = 0; i < PER; i += 4) {
      const float4 x =
          *reinterpret_cast<const float4*>(st_wv + (size_t)(b * 2) * T + (i / 4) * THREADS * 4 + tid * 4);
      wt[i] = x.x; wt[i + 1] = x.y; wt[i + 2] = x.z; wt[i + 3] = x.w;
      acc[i] = acc[i + 1] = acc[i + 2] = acc[i + 3] = 0.f;
    }
    for (int gi = 0; gi < groups && !failed; ++gi, ++sc) {
      const int s = sc % STAGES;
      if (!tc::mbar_wait(&full[s], (sc / STAGES) & 1, abortp, status, ERR_META_CONSUMER)) {
        failed = true;
        break;
      }
      const int cnt = min(G, P - gi * G);
      for (int u = 0; u < cnt; ++u) {                       // ascending j
#pragma unroll
        for (int i = 0; i < PER; i += 4) {
          const float4 x = *reinterpret_cast<const float4*>(st_rep + ((size_t)s * G + u) * T +
                                                            (i / 4) * THREADS * 4 + tid * 4);
          acc[i] += x.x - wt[i];
          acc[i + 1] += x.y - wt[i + 1];
          acc[i + 2] += x.z - wt[i + 2];
          acc[i + 3] += x.w - wt[i + 3];
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive_plain(&empty[s]);
    }
    // the result buffers of the tile before last must have been read by their stores
    if (tid == 0) bulk_wait_read_all();
    if (consumers_any(failed, THREADS)) break;
#pragma unroll
    for (int i = 0; i < PER; i += 4) {
      float4 vt = make_float4(0.f, 0.f, 0.f, 0.f);
      if (read_v)
        vt = *reinterpret_cast<const float4*>(st_wv + (size_t)(b * 2 + 1) * T +
                                              (i / 4) * THREADS * 4 + tid * 4);
      float4 vn, wn;
      vn.x = fmaf(mu, vt.x, zeta * (acc[i] * inv_p));
      vn.y = fmaf(mu, vt.y, zeta * (acc[i + 1] * inv_p));
      vn.z = fmaf(mu, vt.z, zeta * (acc[i + 2] * inv_p));
      vn.w = fmaf(mu, vt.w, zeta * (acc[i + 3] * inv_p));
      wn.x = wt[i] + vn.x; wn.y = wt[i + 1] + vn.y; wn.z = wt[i + 2] + vn.z; wn.w = wt[i + 3] + vn.w;
      *reinterpret_cast<float4*>(st_out + (size_t)(b * 2) * T + (i / 4) * THREADS * 4 + tid * 4) = wn;
      *reinterpret_cast<float4*>(st_out + (size_t)(b * 2 + 1) * T + (i / 4) * THREADS * 4 + tid * 4) = vn;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive_plain(&wv_empty[b]);
    tc::fence_proxy_async();
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
    if (tid == 0) {
      bulk_store(w + t * T, st_out + (size_t)(b * 2) * T, T * 4);
      bulk_store(v + t * T, st_out + (size_t)(b * 2 + 1) * T, T * 4);
      if (bcast)
        for (int j = 0; j < P; ++j)
          bulk_store(rep + (size_t)j * stride + t * T, st_out + (size_t)(b * 2) * T, T * 4);
      bulk_commit();
    }
  }
  if (tid == 0) bulk_wait_read_all();
  // the ragged end of the vector: fewer than T elements, by the last block's consumers
  if (blockIdx.x == gridDim.x - 1) {
    const int64_t i0 = n_tiles * T;
    const int64_t rest4 = (n - i0) >> 2;
    for (int64_t q = tid; q < rest4; q += THREADS) {
      const int64_t i = i0 + 4 * q;
      const float4 wt = *reinterpret_cast<const float4*>(w + i);
      float4 vt = make_float4(0.f, 0.f, 0.f, 0.f);
      if (read_v) vt = *reinterpret_cast<const float4*>(v + i);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int j = 0; j < P; ++j)
        acc4(acc, sub4(*reinterpret_cast<const float4*>(rep + (size_t)j * stride + i), wt));
      float4 vn, wn;
      vn.x = fmaf(mu, vt.x, zeta * (acc.x * inv_p));
      vn.y = fmaf(mu, vt.y, zeta * (acc.y * inv_p));
      vn.z = fmaf(mu, vt.z, zeta * (acc.z * inv_p));
      vn.w = fmaf(mu, vt.w, zeta * (acc.w * inv_p));
      wn.x = wt.x + vn.x; wn.y = wt.y + vn.y; wn.z = wt.z + vn.z; wn.w = wt.w + vn.w;
      *reinterpret_cast<float4*>(v + i) = vn;
      *reinterpret_cast<float4*>(w + i) = wn;
      if (bcast)
        for (int j = 0; j < P; ++j) *reinterpret_cast<float4*>(rep + (size_t)j * stride + i) = wn;
    }
    if (tid < (n & 3))
      meta_scalar(rep, stride, w, v, P, (n & ~(int64_t)3) + tid, mu, zeta, inv_p, read_v != 0,
                  bcast != 0);
  }
}

// The opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the kernel.
template <int T, int G, int STAGES, int THREADS>
cudaError_t launch_bulk(mavg_ctx* c, float mu, float zeta, float inv_p, int read_v, int bcast) {
  const size_t smem = ((size_t)STAGES * G * T + 8 * (size_t)T) * sizeof(float);
  static uint64_t attr_set[4] = {0, 0, 0, 0};   // one bit per device ordinal (< 256)
  const int dev = c->device & 255;
  if (!(attr_set[dev >> 6] >> (dev & 63) & 1)) {
    cudaError_t e = cudaFuncSetAttribute(k_meta_update_bulk<T, G, STAGES, THREADS>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set[dev >> 6] |= (uint64_t)1 << (dev & 63);
  }
  const int64_t n_tiles = c->cfg.n / T;
  const int grid = (int)(n_tiles < c->sm_count ? n_tiles : c->sm_count);
  k_meta_update_bulk<T, G, STAGES, THREADS><<<grid, THREADS + 32, smem, c->stream>>>(
      c->buf.replicas, c->buf.replica_stride, c->buf.global_w, c->buf.momentum, c->cfg.P, c->cfg.n,
      mu, zeta, inv_p, read_v, bcast, (int*)ws_ptr(c, c->ws.status));
  return cudaGetLastError();
}

int grid_for(const mavg_ctx* c, int64_t work_items, int threads, int blocks_per_sm) {
  int64_t need = (work_items + threads - 1) / threads;
  int64_t cap = (int64_t)c->sm_count * blocks_per_sm;
  if (need < 1) need = 1;
  return (int)(need < cap ? need : cap);
}

}  // namespace

cudaError_t launch_broadcast(mavg_ctx* c, bool zero_v, bool force_copies) {
  const int64_t n = c->cfg.n;
  const bool copies = force_copies || !c->cfg.defer_broadcast;
  c->replicas_materialized = copies;
  if (!copies && !zero_v) return cudaSuccess;
  int grid = grid_for(c, n >> 2, 256, 8);
  prof_begin(c, MAVG_K_BROADCAST);
  k_broadcast<<<grid, 256, 0, c->stream>>>(c->buf.replicas, c->buf.replica_stride,
                                           c->buf.global_w, c->buf.momentum, copies ? c->cfg.P : 0,
                                           n, zero_v ? 1 : 0);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_meta_update(mavg_ctx* c) {
  const int64_t n = c->cfg.n;
  const int P = c->cfg.P;
  const float mu = c->cfg.mu, zeta = c->cfg.block_lr;
  const float inv_p = 1.0f / (float)P;
  const int read_v = mu != 0.f ? 1 : 0;
  const int bcast = c->cfg.defer_broadcast ? 0 : 1;
  c->replicas_materialized = bcast != 0;
  // A replica set that fits in L2 is about to be re-read by the next round's first local step:
  // it takes the register kernel with plain stores, which leaves it there (and writes the bf16
  // copy of w~ on the way where a tensor-core handle asks for it).  Larger sets go through the
  // bulk-copy kernel, whose ring shape is picked by P (measured at n = 11.2 M on a B200: each of
  // the three is the fastest, by 2-8 %, in its range; the register kernel with evict-first
  // stores was 3-8 % behind them at every P from 4 to 64).
  const bool big = (size_t)P * (size_t)n * 4 > c->l2_bytes / 2;
  prof_begin(c, MAVG_K_META);
  cudaError_t e = cudaSuccess;
  c->shadow_fresh = false;
  if (big && n >= (int64_t)4096 * c->sm_count * 4) {
    if (P <= 4) e = launch_bulk<2048, 4, 3, 256>(c, mu, zeta, inv_p, read_v, bcast);
    else if (P <= 8 || P >= 24) e = launch_bulk<2048, 6, 2, 512>(c, mu, zeta, inv_p, read_v, bcast);
    else e = launch_bulk<4096, 3, 2, 512>(c, mu, zeta, inv_p, read_v, bcast);
  } else {
    int grid = grid_for(c, n >> 2, 256, 8);
    float* rep = c->buf.replicas;
    float* w = c->buf.global_w;
    float* v = c->buf.momentum;
    if (big)
      k_meta_update<8, true><<<grid, 256, 0, c->stream>>>(rep, c->buf.replica_stride, w, v, P,
                                                          n, mu, zeta, inv_p, read_v, bcast);
    else if (c->shadow.dst) {
      k_meta_update<8, false, true><<<grid, 256, 0, c->stream>>>(rep, c->buf.replica_stride, w, v, P,
                                                                 n, mu, zeta, inv_p, read_v, bcast,
                                                                 c->shadow);
      c->shadow_fresh = true;
    } else
      k_meta_update<8, false><<<grid, 256, 0, c->stream>>>(rep, c->buf.replica_stride, w, v, P,
                                                           n, mu, zeta, inv_p, read_v, bcast);
    e = cudaGetLastError();
  }
  prof_end(c);
  return e;
}

}  // namespace mavg
