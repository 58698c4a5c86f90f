// Tensor-core MLP learner step: the three matrix products of every layer run on tcgen05 with
// TMA-fed shared-memory operands and the accumulator in tensor memory.  This file holds the
// forward and dgrad kernel and the schedule of a step; the weight-gradient kernel, which carries
// the SGD step, is in wgrad_tc.cu.
//
// Every product is arranged so that the 128-row MMA dimension is a feature dimension and the
// batch (16..256 rows) is the MMA's N or K:
//   forward   Z^T[out, B]  = W[out, in]    . A[B, in]^T        contraction over in
//   dgrad     dA^T[in, B]  = W^T[in, out]  . dZ[B, out]^T      contraction over out (W^T = W read MN-major)
//   wgrad     dW[out, in]  = dZ^T[out, B]  . A^T[in, B]^T      contraction over the batch
// Activations and dZ are kept in both orientations ([B, f] and [f, B]; the producing epilogues
// write both) so that they are K-major wherever they are an operand.  The weights have one bf16
// copy, [out, in]: forward reads it K-major, dgrad reads the same tiles MN-major.  fp32 master
// weights take the SGD step of Algorithm 1 in the wgrad kernel, which also refreshes the bf16
// copy.
// When a layer has too few output tiles to fill the GPU, forward and dgrad split the contraction
// over several blocks; each writes an fp32 partial tile and the block that finishes last adds
// the partials in ascending split order (so the result does not depend on which block that is).
// That block -- or the only block, when there is no split -- applies the layer's tail in the
// same kernel: bias + ReLU, or the ReLU mask with the bias step of the layer below, or for the
// last layer the softmax cross-entropy loss, dZ_L and the last bias step.
#include <cuda.h>

#include <algorithm>

#include "mlp.cuh"
#include "tc_ptx.cuh"
#include "wgrad_tc.cuh"

namespace mavg {
namespace {

using namespace tc;

constexpr int kBM = 128;        // MMA M (rows of operand A per tile)
constexpr int kBK = 64;         // contraction elements per pipeline stage (128 bytes of bf16)
constexpr int kThreads = 320;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
constexpr int kMaxStages = 8;
constexpr int kATileBytes = kBM * kBK * 2;

enum { EPI_FWD_HIDDEN = 0, EPI_FWD_LAST = 1, EPI_DGRAD = 2 };
enum { ERR_PRODUCER = 11, ERR_MMA = 12, ERR_EPILOGUE = 13 };

struct TcArgs {
  int M, N;                 // valid rows of A and of B
  int BN;                   // N tile: multiple of 16, <= 256
  int m_tiles, n_tiles, splits, kb_per_split, nkb, stages;
  int a_batched, b_batched; // 0: the operand is shared by all learners
  int a_mn;                 // 1: A is read MN-major from a [K rows, M contiguous] array (dgrad: W itself)
  int P;
  uint32_t tmem_cols;
  // forward / dgrad: A rows are features m (M of them), B rows the batch (N = B of them)
  float* part;              // split partials, part[((split*P + p)*N + n)*M + m]
  int* counters;            // one per (p, m_tile); zero between launches
  float* bias_rep;          // fp32 masters; the bias this kernel reads (forward) or steps (dgrad,
  int64_t bias_off;         // last layer) is at bias_rep[p*rep_stride + bias_off + m]
  const float* bias_in;     // where the bias is read: bias_in[p*bias_in_stride + bias_off + m], the
  int64_t bias_in_stride;   // same place, or w~ (stride 0) at the first step of a round
  __nv_bfloat16* out_bm;    // [P, B, M]  relu(z) (forward) or dZ (dgrad)
  __nv_bfloat16* out_mb;    // [P, M, B]  the same, transposed
  const __nv_bfloat16* mask_mb;  // dgrad: forward activation [P, M, B] whose sign gates dZ
  // last layer (M = classes <= 32): loss, dZ_L and the bias step
  const int32_t* labels;    // [P*B]
  float* loss_out;          // loss_out[p*loss_stride]
  int loss_stride;
  __nv_bfloat16* dz_bm;     // [P, B, cpad]
  int cpad;
  __nv_bfloat16* dz_mb;     // [P, M, B]
  int64_t rep_stride;
  float gamma;
  MomArgs mom;              // learner momentum of the bias this kernel steps (slots laid out like bias_rep)
  int* status;
};

// Synchronises the 8 epilogue warps (256 threads) without the producer and MMA warps.
__device__ __forceinline__ void epilogue_barrier() {
  asm volatile("bar.sync 1, 256;" ::: "memory");
}

// 32 accumulator columns starting at c0 for this warp's 32 lanes (16 when the tile ends there;
// the rest reads as zero).  Returns the number of valid columns.  Warp-collective.
__device__ __forceinline__ int load_acc_chunk(uint32_t lane_addr, int c0, int BN, float (&z)[32]) {
  uint32_t r[32];
  if (c0 + 32 <= BN) {
    tmem_ld_32x32(lane_addr + (uint32_t)c0, r);
  } else {                                   // BN is a multiple of 16
    uint32_t h[16];
    tmem_ld_16cols(lane_addr + (uint32_t)c0, h);
#pragma unroll
    for (int j = 0; j < 16; ++j) { r[j] = h[j]; r[16 + j] = 0u; }
  }
  tmem_ld_wait();
#pragma unroll
  for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(r[j]);
  return min(32, BN - c0);
}

// MINB = 2 caps the registers so that two blocks fit an SM (used when a launch has more blocks
// than SMs; costs a few spills in the tail), MINB = 1 leaves the compiler free.
template <int EPI, int MINB>
__global__ void __launch_bounds__(kThreads, MINB)
k_tc_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
          const TcArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int last_flag;
  __shared__ float colsum[2][kBM];

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stage_bytes = kATileBytes + g.BN * kBK * 2;
  const int stages = g.stages;

  const int split = blockIdx.x % g.splits;
  const int tile = blockIdx.x / g.splits;
  const int n_tile = tile % g.n_tiles, m_tile = tile / g.n_tiles;
  const int p = blockIdx.y;
  const int m0 = m_tile * kBM, n0 = n_tile * g.BN;
  const int kb0 = split * g.kb_per_split;
  const int kb1 = min(g.nkb, kb0 + g.kb_per_split);
  const int count = kb1 - kb0;

  grid_launch_dependents();   // the next kernel may begin its own set-up early
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&acc_bar, 1);
    abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, g.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  // Everything above touched only this block's own shared and tensor memory.  When the launch
  // allowed it, that much ran while the previous kernel of the stream was still finishing; from
  // here on its results are read, so wait for it to complete (returns at once otherwise).
  grid_dependency_wait();
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int i = 0; i < count; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&empty_bar[s], (u & 1) ^ 1, abortp, g.status, ERR_PRODUCER)) break;
        uint8_t* sa = smem + (size_t)s * stage_bytes;
        mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
        if (g.a_mn) {     // two 64-wide halves of the M range, each 64 K-rows of 128 bytes
          tma_load_3d(sa, &tmA, &full_bar[s], m0, (kb0 + i) * kBK, g.a_batched ? p : 0);
          tma_load_3d(sa + kATileBytes / 2, &tmA, &full_bar[s], m0 + 64, (kb0 + i) * kBK,
                      g.a_batched ? p : 0);
        } else {
          tma_load_3d(sa, &tmA, &full_bar[s], (kb0 + i) * kBK, m0, g.a_batched ? p : 0);
        }
        tma_load_3d(sa + kATileBytes, &tmB, &full_bar[s], (kb0 + i) * kBK, n0,
                    g.b_batched ? p : 0);
        issued = i + 1;
      }
      if (*abortp) {
        // give the copies already issued a bounded chance to land before the block retires
        for (int i = max(0, issued - stages); i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&full_bar[i % stages], (i / stages) & 1))
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, g.BN, g.a_mn);
      bool ok = true;
      for (int i = 0; i < count; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&full_bar[s], u & 1, abortp, g.status, ERR_MMA)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        const uint64_t adesc = g.a_mn ? smem_desc_mn_sw128(sa) : smem_desc_k_sw128(sa);
        const uint64_t bdesc = smem_desc_k_sw128(sa + kATileBytes);
        // per MMA (16 K-elements) a K-major tile advances 32 bytes inside its 128-byte rows, an
        // MN-major tile 16 rows of 128 bytes; descriptor addresses count 16-byte units
        const uint32_t a_step = g.a_mn ? (16 * 128) >> 4 : 2;
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)
          umma_bf16(tmem_base, adesc + a_step * k, bdesc + 2 * k, idesc, (uint32_t)((i | k) != 0));
        umma_commit(&empty_bar[s]);
      }
      if (ok) umma_commit(&acc_bar);
    }
    __syncwarp();
  } else {
    // 8 epilogue warps: warp (q, half) owns TMEM lanes [32q, 32q+32) -- the only lanes a warp
    // with (warp index mod 4) == q may read -- and every second 32-column chunk.
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    const int row = q * 32 + lane;
    // Operands of the tail that do not depend on the accumulator are fetched while the main loop
    // is still running: the bias (read by the forward tails, stepped by the dgrad tail), the
    // first mask chunk (dgrad) and the label of this thread's batch row (last layer).
    float* bias = g.bias_rep + (size_t)p * g.rep_stride + g.bias_off;
    const float* bias_in = g.bias_in + (size_t)p * g.bias_in_stride + g.bias_off;
    const bool m_ok_pre = m0 + row < g.M;
    const float bias_pre = (m_ok_pre && (EPI != EPI_DGRAD || half == 0)) ? bias_in[m0 + row] : 0.f;
    uint4 mk[4] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0),
                   make_uint4(0, 0, 0, 0)};
    auto load_mask = [&](int c0, uint4 (&dst)[4]) {
      if (!m_ok_pre || c0 >= g.BN) return;
      const uint4* msrc = reinterpret_cast<const uint4*>(
          g.mask_mb + ((size_t)p * g.M + m0 + row) * g.N + n0 + c0);
      if (n0 + c0 + 32 <= g.N) {               // whole chunk inside the batch: 4 loads in flight
#pragma unroll
        for (int v = 0; v < 4; ++v) dst[v] = msrc[v];
      } else {
#pragma unroll
        for (int v = 0; v < 4; ++v)
          dst[v] = n0 + c0 + v * 8 < g.N ? msrc[v] : make_uint4(0, 0, 0, 0);
      }
    };
    // (only in the one-block-per-SM build: the register-capped build has no room to hold it)
    if (EPI == EPI_DGRAD) load_mask(half * 32, mk);
    int label_pre = 0;
    if (EPI == EPI_FWD_LAST && ew * 32 + lane < g.N)
      label_pre = g.labels[(size_t)p * g.N + ew * 32 + lane];
    const bool ok = mbar_wait(&acc_bar, 0, abortp, g.status, ERR_EPILOGUE);
    tc_fence_after_sync();
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    {
      // forward / dgrad: feature m per lane, the batch along the columns (the dgrad and last-layer
      // tails need the whole batch in one tile: n_tiles == 1 there)
      const int m = m0 + row;
      const bool m_ok = m < g.M;
      bool finisher = ok;
      if (MINB == 1 && g.splits > 1) {   // the register-capped build is never used with a split
        if (ok) {
          float* dst = g.part + ((size_t)(split * g.P + p) * g.N) * g.M + m;
          for (int c0 = half * 32; c0 < g.BN; c0 += 64) {
            float z[32];
            const int ncols = load_acc_chunk(lane_addr, c0, g.BN, z);
            if (m_ok) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < ncols && n0 + c0 + j < g.N) dst[(size_t)(n0 + c0 + j) * g.M] = z[j];
            }
          }
        }
        // the block that publishes the last of the `splits` partials of this tile finishes it
        __threadfence();
        epilogue_barrier();
        if (ew == 0 && lane == 0) {
          int* ctr = g.counters + (p * g.m_tiles + m_tile) * g.n_tiles + n_tile;
          const int old = ok ? atomicAdd(ctr, 1) : -1;
          const int last = old == g.splits - 1;
          if (last) *ctr = 0;
          __threadfence();
          last_flag = last;
        }
        epilogue_barrier();
        finisher = last_flag != 0;
      }
      if (finisher) {
        const float my_bias = EPI != EPI_DGRAD ? bias_pre : 0.f;
        float dsum = 0.f;
        float* lg = reinterpret_cast<float*>(smem);          // last layer: logits [N][M]
        for (int c0 = half * 32; c0 < g.BN; c0 += 64) {
          float z[32];
          int ncols;
          if (MINB != 1 || g.splits == 1) {
            ncols = load_acc_chunk(lane_addr, c0, g.BN, z);
          } else {
            ncols = min(32, g.BN - c0);
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = 0.f;
            if (m_ok) {
              const int nvalid = min(ncols, g.N - n0 - c0);
#pragma unroll 2
              for (int sp = 0; sp < g.splits; ++sp) {        // ascending split order
                const float* src = g.part + ((size_t)(sp * g.P + p) * g.N + n0 + c0) * g.M + m;
                float t[32];
                if (nvalid == 32) {                          // all loads in flight together
#pragma unroll
                  for (int j = 0; j < 32; ++j) t[j] = __ldcg(src + (size_t)j * g.M);
                } else {
#pragma unroll
                  for (int j = 0; j < 32; ++j)
                    t[j] = __ldcg(src + (size_t)min(j, max(nvalid - 1, 0)) * g.M);
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) z[j] += j < nvalid ? t[j] : 0.f;
              }
            }
          }
          if (EPI == EPI_FWD_LAST) {
            if (m_ok) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < ncols && n0 + c0 + j < g.N) lg[(n0 + c0 + j) * g.M + m] = z[j] + my_bias;
            }
          } else {
            uint32_t hp[16];                                  // 32 bf16 results, packed
            if (EPI == EPI_DGRAD) {
              uint4 mkn[4] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0),
                              make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
              load_mask(c0 + 64, mkn);                        // next chunk, used one iteration on
              const __nv_bfloat16* mh = reinterpret_cast<const __nv_bfloat16*>(mk);
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const bool live = j < ncols && n0 + c0 + j < g.N && __bfloat162float(mh[j]) > 0.f;
                z[j] = live ? z[j] : 0.f;                     // ReLU'(0) = 0
                dsum += z[j];
              }
#pragma unroll
              for (int v = 0; v < 4; ++v) mk[v] = mkn[v];
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float a = z[j] + my_bias;
                z[j] = a > 0.f ? a : 0.f;
              }
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(z[2 * j], z[2 * j + 1]);
              hp[j] = *reinterpret_cast<uint32_t*>(&h2);
            }
            if (m_ok) {
              const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(hp);
              __nv_bfloat16* dbm = g.out_bm + ((size_t)p * g.N + n0 + c0) * g.M + m;
              uint4* dmb = reinterpret_cast<uint4*>(g.out_mb + ((size_t)p * g.M + m) * g.N + n0 + c0);
              if (ncols == 32 && n0 + c0 + 32 <= g.N) {
#pragma unroll
                for (int v = 0; v < 4; ++v)
                  dmb[v] = make_uint4(hp[4 * v], hp[4 * v + 1], hp[4 * v + 2], hp[4 * v + 3]);
#pragma unroll
                for (int j = 0; j < 32; ++j) dbm[(size_t)j * g.M] = hh[j];
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (j < ncols && n0 + c0 + j < g.N) dbm[(size_t)j * g.M] = hh[j];
#pragma unroll
                for (int v = 0; v < 4; ++v)
                  if (v * 8 < ncols && n0 + c0 + v * 8 < g.N)
                    dmb[v] = make_uint4(hp[4 * v], hp[4 * v + 1], hp[4 * v + 2], hp[4 * v + 3]);
              }
            }
          }
        }
        if (EPI == EPI_DGRAD) {
          // bias step of the layer below: b[m] -= gamma * sum_b dZ[b, m]; the two warps that
          // share a row add their column sums in a fixed order
          colsum[half][row] = dsum;
          epilogue_barrier();
          if (half == 0 && m_ok) {
            float* ub = g.mom.u ? g.mom.u + (size_t)p * g.mom.u_stride + g.bias_off + m : nullptr;
            local_update(bias + m, bias_pre, ub, g.mom.read_u, colsum[0][row] + colsum[1][row],
                         g.gamma, g.mom.beta);
          }
        }
        if (EPI == EPI_FWD_LAST) {
          // softmax cross-entropy on the block's [N, M] logits: thread t takes batch row t
          float* dzs = lg + g.N * g.M;
          float* lossp = dzs + g.N * g.M;
          epilogue_barrier();
          const int t = ew * 32 + lane;
          const int C = g.M;
          if (t < g.N) {
            const float* zr = lg + t * C;
            float mx = zr[0];
            for (int c = 1; c < C; ++c) mx = fmaxf(mx, zr[c]);
            float se = 0.f;
            for (int c = 0; c < C; ++c) se += expf(zr[c] - mx);
            const float lse = mx + logf(se);
            const int yb = label_pre;
            lossp[t] = lse - zr[yb];
            const float inv_b = 1.0f / (float)g.N;
            for (int c = 0; c < C; ++c) {
              const float gr = (expf(zr[c] - lse) - (c == yb ? 1.f : 0.f)) * inv_b;
              dzs[t * C + c] = gr;
              const __nv_bfloat16 gq = __float2bfloat16_rn(gr);
              g.dz_bm[((size_t)p * g.N + t) * g.cpad + c] = gq;
              g.dz_mb[((size_t)p * C + c) * g.N + t] = gq;
            }
          }
          epilogue_barrier();
          // loss: every warp adds its 32 rows, thread 0 the warps' sums; bias gradient of class c:
          // a warp adds the rows lane, lane + 32, ... and then its lanes, in a fixed order
          {
            float sl = t < g.N ? lossp[t] : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sl += __shfl_xor_sync(0xffffffffu, sl, o);
            if (lane == 0) colsum[0][ew] = sl;
            for (int c = ew; c < C; c += 8) {
              float sb = 0.f;
              for (int b = lane; b < g.N; b += 32) sb += dzs[b * C + c];
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) sb += __shfl_xor_sync(0xffffffffu, sb, o);
              if (lane == 0) {
                float* ub = g.mom.u ? g.mom.u + (size_t)p * g.mom.u_stride + g.bias_off + c : nullptr;
                local_update(bias + c, bias_in[c], ub, g.mom.read_u, sb, g.gamma, g.mom.beta);
              }
            }
          }
          epilogue_barrier();
          if (t == 0) {
            float sl = 0.f;
            const int nw = (g.N + 31) / 32;
            for (int w = 0; w < nw; ++w) sl += colsum[0][w];
            g.loss_out[(size_t)p * g.loss_stride] = sl / (float)g.N;
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, g.tmem_cols);
}

// bf16 copy of the global model w~ (shared by all learners at the first step of a round, when
// every replica equals w~).  One launch per layer; grid-stride over the layer's weights.
__global__ void __launch_bounds__(256)
k_shadow_from_global(const float* __restrict__ w, int64_t w_off, int64_t total,
                     __nv_bfloat16* __restrict__ w16, int64_t sh_off) {
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x)
    w16[sh_off + t] = __float2bfloat16_rn(w[w_off + t]);
}

// ---------------------------------------------------------------------------------- host side
size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct TcLayout {
  int L;
  int cpad;                                  // last layer's dZ row length (multiple of 8)
  int64_t n16;                               // elements per bf16 copy row
  int64_t sh_off[MAVG_MAX_LAYERS];
  size_t xg[2], xt[2];                       // gathered batch, two buffers used by alternate steps
  size_t act[MAVG_MAX_LAYERS + 1], act_t[MAVG_MAX_LAYERS + 1];
  size_t dz[MAVG_MAX_LAYERS + 1], dz_t[MAVG_MAX_LAYERS + 1];
  size_t part, part_bytes;
  size_t counters, counters_bytes;
  size_t w16, w16g;
  size_t end;
};

struct GemmPlan { int m_tiles, n_tiles, splits, kb_per_split, nkb, BN, stages, two_per_sm; uint32_t tmem_cols; };

// Forward / dgrad plan.  To fill the GPU the batch may be cut into column tiles (`tile_n`: only
// the hidden-layer forward can, its tail needs no sum over the batch) and, if blocks are still
// few and the contraction long, the contraction is split; a block never gets fewer than 8 slabs
// (512 elements), below which the split's fix-up costs more than it saves.
GemmPlan plan_partial(int M, int N, int K, int P, int sm_count, bool tile_n) {
  GemmPlan g{};
  g.BN = (N + 15) / 16 * 16;
  g.m_tiles = (M + kBM - 1) / kBM;
  g.n_tiles = 1;
  g.nkb = (K + kBK - 1) / kBK;
  const int enough = sm_count - sm_count / 5;   // ~80 % of the SMs busy counts as full
  if (tile_n)
    while (g.m_tiles * g.n_tiles * P < enough && g.BN % 64 == 0) {
      g.BN /= 2;
      g.n_tiles *= 2;
    }
  int tiles = g.m_tiles * g.n_tiles * P;
  int want = tiles >= enough ? 1 : (sm_count + tiles - 1) / tiles;
  if (want > g.nkb / 8) want = g.nkb / 8;
  if (want < 1) want = 1;
  g.kb_per_split = (g.nkb + want - 1) / want;
  g.splits = (g.nkb + g.kb_per_split - 1) / g.kb_per_split;
  int stage_bytes = kATileBytes + g.BN * kBK * 2;
  // more blocks than SMs: two blocks share an SM, so that one block's set-up and tail overlap
  // the other's main loop; otherwise one block takes the whole shared memory
  g.two_per_sm = (g.splits == 1 && g.m_tiles * g.n_tiles * P > sm_count) ? 1 : 0;
  const int budget = g.two_per_sm ? 104 * 1024 : 200 * 1024;
  g.stages = budget / stage_bytes;
  if (g.stages > kMaxStages) g.stages = kMaxStages;
  if (g.stages > g.kb_per_split) g.stages = g.kb_per_split < 2 ? 2 : g.kb_per_split;
  g.tmem_cols = 32;
  while ((int)g.tmem_cols < g.BN) g.tmem_cols <<= 1;
  return g;
}

TcLayout make_layout(const mavg_config* cfg, size_t base, int sm_count) {
  TcLayout t{};
  const int L = cfg->n_layers, P = cfg->P, B = cfg->B;
  const size_t rows = (size_t)P * B;
  t.L = L;
  t.cpad = (cfg->dims[L] + 7) / 8 * 8;
  int64_t o16 = 0;
  for (int l = 0; l < L; ++l) {
    t.sh_off[l] = o16;
    o16 += (int64_t)up((size_t)cfg->dims[l] * cfg->dims[l + 1], 64);
  }
  t.n16 = o16;
  size_t off = up(base, 1024);
  auto take = [&](size_t bytes) { size_t r = off; off = up(off + bytes, 1024); return r; };
  for (int i = 0; i < 2; ++i) {
    t.xg[i] = take(rows * cfg->dims[0] * 2);
    t.xt[i] = take(rows * cfg->dims[0] * 2);
  }
  int max_m_tiles = 1;
  for (int l = 1; l <= L; ++l) {
    const int d = cfg->dims[l];
    if (l < L) {
      t.act[l] = take(rows * d * 2);
      t.act_t[l] = take(rows * d * 2);
      t.dz[l] = take(rows * d * 2);
    } else {
      t.dz[l] = take(rows * t.cpad * 2);
    }
    t.dz_t[l] = take(rows * d * 2);
    max_m_tiles = std::max(max_m_tiles, 8 * ((d + kBM - 1) / kBM));   // up to 8 column tiles
  }
  size_t pb = 1024;
  for (int l = 1; l <= L; ++l) {
    GemmPlan f = plan_partial(cfg->dims[l], B, cfg->dims[l - 1], P, sm_count, l < L);
    if (f.splits > 1) pb = std::max(pb, (size_t)f.splits * rows * cfg->dims[l] * 4);
    if (l > 1) {
      GemmPlan d = plan_partial(cfg->dims[l - 1], B, cfg->dims[l], P, sm_count, false);
      if (d.splits > 1) pb = std::max(pb, (size_t)d.splits * rows * cfg->dims[l - 1] * 4);
    }
  }
  t.part_bytes = pb;
  t.part = take(pb);
  t.counters_bytes = (size_t)P * max_m_tiles * sizeof(int);
  t.counters = take(t.counters_bytes);
  t.w16 = take((size_t)P * t.n16 * 2);
  t.w16g = take((size_t)t.n16 * 2);
  t.end = off;
  return t;
}

// SM count the plans (and with them the size of the partial buffer) are made for, so that the
// workspace size does not depend on the device that later runs the problem.
constexpr int kPlanSmCount = 148;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  TcLayout lay;
  EncodeTiledFn encode = nullptr;
  // per layer l = 1..L (index l)
  CUtensorMap w[MAVG_MAX_LAYERS + 1], wg[MAVG_MAX_LAYERS + 1];       // [out, in] copies
  CUtensorMap act_in[MAVG_MAX_LAYERS + 1];    // [B, d_{l-1}] input activations of layer l >= 2
  CUtensorMap act_in_t[MAVG_MAX_LAYERS + 1];  // [d_{l-1}, B]
  CUtensorMap x_in[2], x_in_t[2];             // layer 1's input: the two gather buffers
  CUtensorMap dz[MAVG_MAX_LAYERS + 1];        // [B, d_l]
  CUtensorMap dz_t[MAVG_MAX_LAYERS + 1];      // [d_l, B]
  CUtensorMap w_mn[MAVG_MAX_LAYERS + 1], wg_mn[MAVG_MAX_LAYERS + 1];  // [out, in] copies, 64 x 64 boxes
  CUtensorMap w32[MAVG_MAX_LAYERS + 1];       // fp32 masters [out, in]: wgrad loads and stores
  CUtensorMap w32g[MAVG_MAX_LAYERS + 1];      // the same view of w~ (one copy): first-step loads
  CUtensorMap w16_st[MAVG_MAX_LAYERS + 1];    // store view of the bf16 copy
  CUtensorMap u32[MAVG_MAX_LAYERS + 1];       // learner momentum buffers, the masters' view
  bool wgrad_mom = false;                     // the wgrad plans leave room for the u tile
  GemmPlan fwd[MAVG_MAX_LAYERS + 1], dgrad[MAVG_MAX_LAYERS + 1];
  WgradPlan wgrad[MAVG_MAX_LAYERS + 1];
  // side streams and events for the branches of a step that may overlap
  cudaStream_t s_wgrad = nullptr, s_gather = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_wgrad_done = nullptr, ev_gather_done = nullptr,
              ev_x_free[2] = {nullptr, nullptr};
};

// Tensor [batch, rows, inner] with the given strides (in elements) and box inner x box_rows.
bool encode_any(TcState* st, CUtensorMap* m, CUtensorMapDataType dt, int esize, void* ptr,
                int inner, int rows, int batch, int64_t row_stride, int64_t batch_stride,
                int box_inner, int box_rows, CUtensorMapSwizzle swz, std::string* why) {
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)row_stride * esize, (cuuint64_t)batch_stride * esize};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = st->encode(m, dt, 3, ptr, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (why) *why = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return false;
  }
  return true;
}

// bf16 operand of an MMA: 64-element K slabs, 128-byte swizzle.
bool encode_map(TcState* st, CUtensorMap* m, void* ptr, int inner, int rows, int batch,
                int64_t row_stride, int64_t batch_stride, int box_rows, std::string* why) {
  return encode_any(st, m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, inner, rows, batch, row_stride,
                    batch_stride, kBK, box_rows, CU_TENSOR_MAP_SWIZZLE_128B, why);
}

template <int EPI>
cudaError_t launch_gemm(mavg_ctx* c, int cls, const CUtensorMap& a, const CUtensorMap& b,
                        const GemmPlan& pl, TcArgs g) {
  g.BN = pl.BN;
  g.m_tiles = pl.m_tiles;
  g.n_tiles = pl.n_tiles;
  g.splits = pl.splits;
  g.kb_per_split = pl.kb_per_split;
  g.nkb = pl.nkb;
  g.stages = pl.stages;
  g.tmem_cols = pl.tmem_cols;
  g.P = c->cfg.P;
  g.rep_stride = c->buf.replica_stride;
  g.gamma = c->cfg.local_lr;
  g.status = (int*)ws_ptr(c, c->ws.status);
  size_t pipe = (size_t)pl.stages * (kATileBytes + pl.BN * kBK * 2);
  size_t smem = pipe + 1024;
  if (EPI == EPI_FWD_LAST)   // the loss tail reuses the pipeline buffers: logits, dZ, row losses
    smem = std::max(pipe, ((size_t)2 * g.N * g.M + g.N) * sizeof(float)) + 1024;
  dim3 grid((unsigned)(pl.m_tiles * pl.n_tiles * pl.splits), (unsigned)c->cfg.P);
  cudaLaunchConfig_t lc{};
  lc.gridDim = grid;
  lc.blockDim = dim3(kThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  prof_begin(c, cls);
  cudaError_t e = pl.two_per_sm ? cudaLaunchKernelEx(&lc, k_tc_gemm<EPI, 2>, a, b, g)
                                : cudaLaunchKernelEx(&lc, k_tc_gemm<EPI, 1>, a, b, g);
  prof_end(c);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

bool tc_shapes_ok(const mavg_config* cfg, std::string* why) {
  if (cfg->B % 16 != 0 || cfg->B > 256) {
    if (why) *why = "the tensor-core path needs B to be a multiple of 16 and at most 256";
    return false;
  }
  for (int l = 0; l < cfg->n_layers; ++l)
    if (cfg->dims[l] % 8 != 0) {
      if (why) *why = "the tensor-core path needs every layer's input width to be a multiple of 8";
      return false;
    }
  if (cfg->dims[cfg->n_layers] > 32) {
    if (why) *why = "the tensor-core path needs at most 32 classes";
    return false;
  }
  return true;
}

size_t tc_workspace_bytes(const mavg_config* cfg, size_t base, size_t* act_off) {
  *act_off = base;
  return make_layout(cfg, base, kPlanSmCount).end;
}

mavg_status tc_setup(mavg_ctx* c) {
  const mavg_config& cfg = c->cfg;
  TcState* st = new TcState();
  c->mlp = st;
  st->lay = make_layout(&cfg, c->ws.act, kPlanSmCount);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) {
    c->err = "cuTensorMapEncodeTiled is not available from this driver";
    cudaGetLastError();
    return MAVG_ERR_UNSUPPORTED;
  }
  st->encode = (EncodeTiledFn)fn;
  const TcLayout& t = st->lay;
  const int L = cfg.n_layers, P = cfg.P, B = cfg.B;
  char* ws = (char*)c->buf.workspace;
  auto bf = [&](size_t off) { return (void*)(ws + off); };
  std::string why;
  bool ok = true;
  for (int l = 1; l <= L && ok; ++l) {
    const int in = cfg.dims[l - 1], out = cfg.dims[l];
    const int dz_ld = l < L ? out : t.cpad;
    st->fwd[l] = plan_partial(out, B, in, P, kPlanSmCount, l < L);
    st->wgrad_mom = c->buf.learner_u != nullptr;
    st->wgrad[l] = plan_wgrad_stream(out, in, B, P, c->sm_count, st->wgrad_mom);
    if (st->wgrad_mom)
      ok = ok && encode_any(st, &st->u32[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                            c->buf.learner_u + c->layers[l - 1].w_off, in, out, P, in,
                            c->buf.replica_stride, kWgradTileCols, kWgradTileRows,
                            CU_TENSOR_MAP_SWIZZLE_128B, &why);
    __nv_bfloat16* w16 = (__nv_bfloat16*)bf(t.w16) + t.sh_off[l - 1];
    __nv_bfloat16* w16g = (__nv_bfloat16*)bf(t.w16g) + t.sh_off[l - 1];
    ok = ok && encode_map(st, &st->w[l], w16, in, out, P, in, t.n16, kBM, &why);
    ok = ok && encode_map(st, &st->wg[l], w16g, in, out, 1, in, t.n16, kBM, &why);
    ok = ok && encode_map(st, &st->w_mn[l], w16, in, out, P, in, t.n16, 64, &why);
    ok = ok && encode_map(st, &st->wg_mn[l], w16g, in, out, 1, in, t.n16, 64, &why);
    if (l == 1) {
      for (int i = 0; i < 2 && ok; ++i) {
        ok = ok && encode_map(st, &st->x_in[i], bf(t.xg[i]), in, B, P, in, (int64_t)B * in,
                              st->fwd[l].BN, &why);
        ok = ok && encode_map(st, &st->x_in_t[i], bf(t.xt[i]), B, in, P, B, (int64_t)B * in,
                              kWgradTileCols, &why);
      }
    } else {
      ok = ok && encode_map(st, &st->act_in[l], bf(t.act[l - 1]), in, B, P, in, (int64_t)B * in,
                            st->fwd[l].BN, &why);
      ok = ok && encode_map(st, &st->act_in_t[l], bf(t.act_t[l - 1]), B, in, P, B,
                            (int64_t)B * in, kWgradTileCols, &why);
    }
    ok = ok && encode_map(st, &st->dz_t[l], bf(t.dz_t[l]), B, out, P, B, (int64_t)B * out, kBM,
                          &why);
    ok = ok && encode_any(st, &st->w32[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                          c->buf.replicas + c->layers[l - 1].w_off, in, out, P, in,
                          c->buf.replica_stride, kWgradTileCols, kWgradTileRows,
                          CU_TENSOR_MAP_SWIZZLE_128B, &why);
    ok = ok && encode_any(st, &st->w32g[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                          c->buf.global_w + c->layers[l - 1].w_off, in, out, 1, in,
                          c->buf.replica_stride, kWgradTileCols, kWgradTileRows,
                          CU_TENSOR_MAP_SWIZZLE_128B, &why);
    ok = ok && encode_any(st, &st->w16_st[l], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w16, in, out, P,
                          in, t.n16, kWgradTileCols, kWgradTileRows, CU_TENSOR_MAP_SWIZZLE_64B,
                          &why);
    if (l > 1) {
      st->dgrad[l] = plan_partial(in, B, out, P, kPlanSmCount, false);
      ok = ok && encode_map(st, &st->dz[l], bf(t.dz[l]), out, B, P, dz_ld, (int64_t)B * dz_ld,
                            st->dgrad[l].BN, &why);
    }
  }
  if (!ok) {
    c->err = why;
    return MAVG_ERR_CUDA;
  }
  // 227 KB per block in all, of which a few hundred bytes are the kernel's static variables
  constexpr int kMaxDynSmem = 225 * 1024;
  e = cudaSuccess;
  const void* kernels[] = {(const void*)k_tc_gemm<EPI_FWD_HIDDEN, 1>, (const void*)k_tc_gemm<EPI_FWD_HIDDEN, 2>,
                           (const void*)k_tc_gemm<EPI_FWD_LAST, 1>,   (const void*)k_tc_gemm<EPI_FWD_LAST, 2>,
                           (const void*)k_tc_gemm<EPI_DGRAD, 1>,      (const void*)k_tc_gemm<EPI_DGRAD, 2>};
  for (const void* k : kernels)
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  if (e == cudaSuccess) e = wgrad_stream_prepare();
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&st->s_wgrad, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&st->s_gather, cudaStreamNonBlocking);
  cudaEvent_t* evs[] = {&st->ev_fork, &st->ev_wgrad_done, &st->ev_gather_done, &st->ev_x_free[0],
                        &st->ev_x_free[1]};
  for (cudaEvent_t* ev : evs)
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ws + t.counters, 0, t.counters_bytes, c->stream);
  if (e != cudaSuccess) {
    c->err = std::string("tensor-core path set-up: ") + cudaGetErrorString(e);
    cudaGetLastError();   // reported here; do not leave it pending for a later call
    return MAVG_ERR_CUDA;
  }
  return MAVG_OK;
}

void tc_teardown(mavg_ctx* c) {
  TcState* st = (TcState*)c->mlp;
  if (st) {
    if (st->s_wgrad) cudaStreamDestroy(st->s_wgrad);
    if (st->s_gather) cudaStreamDestroy(st->s_gather);
    cudaEvent_t evs[] = {st->ev_fork, st->ev_wgrad_done, st->ev_gather_done, st->ev_x_free[0],
                         st->ev_x_free[1]};
    for (cudaEvent_t ev : evs)
      if (ev) cudaEventDestroy(ev);
  }
  delete st;
  c->mlp = nullptr;
}

cudaError_t tc_refresh_shared_operands(mavg_ctx* c) {
  TcState* st = (TcState*)c->mlp;
  const TcLayout& t = st->lay;
  char* ws = (char*)c->buf.workspace;
  for (int l = 1; l <= c->cfg.n_layers; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    const int64_t total = (int64_t)ly.in * ly.out;
    int grid = (int)std::min<int64_t>((total + 255) / 256, (int64_t)c->sm_count * 8);
    prof_begin(c, MAVG_K_AUX);
    k_shadow_from_global<<<grid, 256, 0, c->stream>>>(c->buf.global_w, ly.w_off, total,
                                                      (__nv_bfloat16*)(ws + t.w16g),
                                                      t.sh_off[l - 1]);
    prof_end(c);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// One local step of all learners.  Dependencies inside a step:
//   gather -> fwd_1 -> ... -> fwd_L (+loss) -> dgrad_L -> ... -> dgrad_2 -> wgrad_1
//   wgrad_l (l >= 2) needs dZ_l and must follow dgrad_l, which still reads W_l; it does not feed
//   anything else of this step, so it runs on a side stream beside the rest of the chain.
//   The gather of the next step touches no weights; it runs on a second side stream into the
//   other of two batch buffers as soon as that buffer's last reader (wgrad_1 of the step before
//   last) is done.
// With `overlap` false (profiled runs) everything is issued in order on the main stream.
cudaError_t tc_step(mavg_ctx* c, int64_t round, int step) {
  TcState* st = (TcState*)c->mlp;
  const TcLayout& t = st->lay;
  const mavg_config& cfg = c->cfg;
  const int B = cfg.B, L = cfg.n_layers, K = cfg.K;
  char* ws = (char*)c->buf.workspace;
  auto bfp = [&](size_t off) { return (__nv_bfloat16*)(ws + off); };
  int32_t* idx = (int32_t*)ws_ptr(c, c->ws.idx);
  int32_t* labels = (int32_t*)ws_ptr(c, c->ws.labels);
  float* losses = (float*)ws_ptr(c, c->ws.losses);
  float* part = (float*)(ws + t.part);
  int* counters = (int*)(ws + t.counters);
  const bool shared_w = c->replicas_equal_global;   // first step after a (re-)broadcast
  const MomArgs mom = mom_args(c, shared_w);
  const bool overlap = !c->profiling;
  const int xb = step & 1;                          // batch buffer of this step
  cudaStream_t main_s = c->stream;
  cudaError_t e;
#define TC_TRY(call) do { if ((e = (call)) != cudaSuccess) { c->stream = main_s; return e; } } while (0)

  // labels and indices are per step as well: they live beside the batch buffer they belong to
  int32_t* idx_b = idx;
  int32_t* labels_b = labels;
  if (step == 1 || !overlap) {
    TC_TRY(launch_sample_gather(c, round, step, idx_b, labels_b, bfp(t.xg[xb]), bfp(t.xt[xb])));
  } else {
    // issued during the previous step on the gather stream
    TC_TRY(cudaStreamWaitEvent(main_s, st->ev_gather_done, 0));
  }

  for (int l = 1; l <= L; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    TcArgs g{};
    g.M = ly.out; g.N = B;
    g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
    g.part = part; g.counters = counters;
    g.bias_rep = c->buf.replicas; g.bias_off = ly.b_off;
    g.bias_in = shared_w ? c->buf.global_w : c->buf.replicas;
    g.bias_in_stride = shared_w ? 0 : c->buf.replica_stride;
    const CUtensorMap& wm = shared_w ? st->wg[l] : st->w[l];
    const CUtensorMap& am = l == 1 ? st->x_in[xb] : st->act_in[l];
    if (l < L) {
      g.out_bm = bfp(t.act[l]); g.out_mb = bfp(t.act_t[l]);
      TC_TRY(launch_gemm<EPI_FWD_HIDDEN>(c, MAVG_K_FWD, wm, am, st->fwd[l], g));
    } else {
      g.labels = labels_b; g.loss_out = losses + (step - 1); g.loss_stride = K;
      g.dz_bm = bfp(t.dz[L]); g.cpad = t.cpad; g.dz_mb = bfp(t.dz_t[L]);
      g.mom = mom;
      TC_TRY(launch_gemm<EPI_FWD_LAST>(c, MAVG_K_FWD, wm, am, st->fwd[l], g));
    }
  }
  // the labels of this step have been consumed: the next step's gather may run now
  if (overlap && step < K) {
    const int nb = (step + 1) & 1;
    TC_TRY(cudaEventRecord(st->ev_fork, main_s));
    TC_TRY(cudaStreamWaitEvent(st->s_gather, st->ev_fork, 0));
    if (step >= 2) TC_TRY(cudaStreamWaitEvent(st->s_gather, st->ev_x_free[nb], 0));
    c->stream = st->s_gather;
    TC_TRY(launch_sample_gather(c, round, step + 1, idx_b, labels_b, bfp(t.xg[nb]), bfp(t.xt[nb])));
    c->stream = main_s;
    TC_TRY(cudaEventRecord(st->ev_gather_done, st->s_gather));
  }

  bool side_used = false;
  for (int l = L; l >= 1; --l) {
    const MlpLayer& ly = c->layers[l - 1];
    if (l > 1) {
      const MlpLayer& below = c->layers[l - 2];
      TcArgs g{};
      g.M = ly.in; g.N = B;
      g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
      g.part = part; g.counters = counters;
      g.bias_rep = c->buf.replicas; g.bias_off = below.b_off;
      g.bias_in = shared_w ? c->buf.global_w : c->buf.replicas;
      g.bias_in_stride = shared_w ? 0 : c->buf.replica_stride;
      g.out_bm = bfp(t.dz[l - 1]); g.out_mb = bfp(t.dz_t[l - 1]);
      g.mask_mb = bfp(t.act_t[l - 1]);
      g.a_mn = 1;
      g.mom = mom;
      TC_TRY(launch_gemm<EPI_DGRAD>(c, MAVG_K_DGRAD, shared_w ? st->wg_mn[l] : st->w_mn[l],
                                    st->dz[l], st->dgrad[l], g));
    }
    const CUtensorMap& bm = l == 1 ? st->x_in_t[xb] : st->act_in_t[l];
    if (overlap && l > 1) {
      TC_TRY(cudaEventRecord(st->ev_fork, main_s));
      TC_TRY(cudaStreamWaitEvent(st->s_wgrad, st->ev_fork, 0));
      c->stream = st->s_wgrad;
      TC_TRY(launch_wgrad_stream(c, st->wgrad[l], st->dz_t[l], bm, st->w32[l], st->w16_st[l],
                                 shared_w ? &st->w32g[l] : nullptr, &st->u32[l], mom));
      c->stream = main_s;
      side_used = true;
    } else {
      TC_TRY(launch_wgrad_stream(c, st->wgrad[l], st->dz_t[l], bm, st->w32[l], st->w16_st[l],
                                 shared_w ? &st->w32g[l] : nullptr, &st->u32[l], mom));
    }
  }
  if (overlap) {
    TC_TRY(cudaEventRecord(st->ev_x_free[xb], main_s));     // wgrad_1 was the buffer's last reader
    if (side_used) {
      TC_TRY(cudaEventRecord(st->ev_wgrad_done, st->s_wgrad));
      TC_TRY(cudaStreamWaitEvent(main_s, st->ev_wgrad_done, 0));
    }
  }
#undef TC_TRY
  return cudaSuccess;
}

}  // namespace mavg
