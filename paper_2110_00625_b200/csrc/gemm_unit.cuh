// One output tile of a forward or dgrad product on tcgen05, with the layer's tail fused: the
// roles (TMA producer, MMA issuer, epilogue warps) of a block that already has its barriers
// initialised and its tensor memory allocated.  Used by the one-tile-per-block kernel and the
// cluster-split kernel of mlp_tc.cu.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace mavg {
namespace gemm {

using namespace tc;

constexpr int kBM = 128;        // MMA M (rows of operand A per tile)
constexpr int kBK = 64;         // contraction elements per pipeline stage (128 bytes of bf16)
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


// Barriers and small scratch of one block, in static shared memory.
struct GemmShared {
  uint64_t full_bar[kMaxStages];
  uint64_t empty_bar[kMaxStages];
  uint64_t acc_bar;
  uint64_t recv_bar;          // cluster split: arrivals of the other blocks' partial tiles
  uint32_t tmem_slot;
  int abort_flag;
  int last_flag;
  float colsum[2][kBM];
};

// Barrier set-up of one tile (one thread): every barrier at phase 0.
__device__ __forceinline__ void gemm_init_barriers(GemmShared& sh, int stages) {
  for (int s = 0; s < stages; ++s) {
    mbar_init(&sh.full_bar[s], 1);
    mbar_init(&sh.empty_bar[s], 1);
  }
  mbar_init(&sh.acc_bar, 1);
}

// The tile with linear index bx (split fastest, then column tile, then row tile) of learner p.
// Warp 0 is the producer, warp 1 the MMA issuer, warps 2-9 the epilogue; further warps return at
// once.  smem: the 1024-byte aligned pipeline buffer.  ALLOW_SPLIT: compile the path that splits
// the contraction over several blocks (g.splits > 1).  All threads of the block must have passed
// a barrier after gemm_init_barriers, and must pass one again before the pipeline buffer or the
// accumulator columns are reused.  A block that runs several tiles keeps using the same
// barriers: it0 is the number of pipeline slabs its earlier tiles went through (with the same
// g.stages) and acc_phase the number of earlier tiles, which fix the barrier phases to wait for.
//
// CLUSTER (hidden-layer forward only): the g.splits blocks that share an output tile form a
// thread-block cluster (rank = split index).  Each accumulates the whole 128 x BN tile over its
// part of the contraction, BN = 32 * g.splits; block r finishes the columns [32 r, 32 r + 32): the
// others write their partial sums of those columns into its shared memory (`recv`, behind the
// pipeline buffer: [splits][128 rows][32] fp32, slot = sender's rank) and arrive on its recv_bar,
// and it adds the partials in ascending rank order.  An SM then takes in 1/splits of the weight
// tile's bytes instead of all of them for a quarter of the batch.
template <int EPI, bool ALLOW_SPLIT, bool CLUSTER = false>
__device__ __forceinline__ void gemm_tile(const CUtensorMap& tmA, const CUtensorMap& tmB,
                                          const TcArgs& g, int bx, int p, uint8_t* smem,
                                          GemmShared& sh, uint32_t tmem_base, uint32_t it0 = 0,
                                          uint32_t acc_phase = 0) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stage_bytes = kATileBytes + g.BN * kBK * 2;
  const int stages = g.stages;
  const int split = bx % g.splits;
  const int tile = bx / g.splits;
  const int n_tile = tile % g.n_tiles, m_tile = tile / g.n_tiles;
  const int m0 = m_tile * kBM, n0 = n_tile * g.BN;
  const int kb0 = split * g.kb_per_split;
  const int kb1 = min(g.nkb, kb0 + g.kb_per_split);
  const int count = kb1 - kb0;
  volatile int* abortp = &sh.abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int i = 0; i < count; ++i) {
        const int s = (it0 + i) % stages, u = (it0 + i) / stages;
        if (!mbar_wait(&sh.empty_bar[s], (u & 1) ^ 1, abortp, g.status, ERR_PRODUCER)) break;
        uint8_t* sa = smem + (size_t)s * stage_bytes;
        mbar_arrive_expect_tx(&sh.full_bar[s], (uint32_t)stage_bytes);
        if (g.a_mn) {     // two 64-wide halves of the M range, each 64 K-rows of 128 bytes
          tma_load_3d(sa, &tmA, &sh.full_bar[s], m0, (kb0 + i) * kBK, g.a_batched ? p : 0);
          tma_load_3d(sa + kATileBytes / 2, &tmA, &sh.full_bar[s], m0 + 64, (kb0 + i) * kBK,
                      g.a_batched ? p : 0);
        } else {
          tma_load_3d(sa, &tmA, &sh.full_bar[s], (kb0 + i) * kBK, m0, g.a_batched ? p : 0);
        }
        tma_load_3d(sa + kATileBytes, &tmB, &sh.full_bar[s], (kb0 + i) * kBK, n0,
                    g.b_batched ? p : 0);
        issued = i + 1;
      }
      if (*abortp) {
        // give the copies already issued a bounded chance to land before the block retires
        for (int i = max(0, issued - stages); i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&sh.full_bar[(it0 + i) % stages], ((it0 + i) / stages) & 1))
            if (global_timer_ns() - t0 > wait_limit_ns(g.status)) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, g.BN, g.a_mn);
      bool ok = true;
      for (int i = 0; i < count; ++i) {
        const int s = (it0 + i) % stages, u = (it0 + i) / stages;
        if (!mbar_wait(&sh.full_bar[s], u & 1, abortp, g.status, ERR_MMA)) { ok = false; break; }
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
        umma_commit(&sh.empty_bar[s]);
      }
      if (ok) umma_commit(&sh.acc_bar);
    }
    __syncwarp();
  } else if (warp < 10) {
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
    const bool ok = mbar_wait(&sh.acc_bar, acc_phase & 1, abortp, g.status, ERR_EPILOGUE);
    tc_fence_after_sync();
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    {
      // forward / dgrad: feature m per lane, the batch along the columns (the dgrad and last-layer
      // tails need the whole batch in one tile: n_tiles == 1 there)
      const int m = m0 + row;
      const bool m_ok = m < g.M;
      bool finisher = ok;
      if (CLUSTER) {
        finisher = false;
        const uint32_t rank = (uint32_t)split;
        float* recv = reinterpret_cast<float*>(smem + (size_t)stages * stage_bytes);
        if (ok) {
          // this warp's chunks that belong to other blocks: into their shared memory
          for (int c0 = half * 32; c0 < g.BN; c0 += 64) {
            const uint32_t dest = (uint32_t)(c0 >> 5);
            if (dest == rank) continue;
            float z[32];
            load_acc_chunk(lane_addr, c0, g.BN, z);
            const uint32_t dst = mapa_u32(smem_u32(recv + ((size_t)rank * kBM + row) * 32), dest);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              st_cluster_f4(dst + 16 * v, z[4 * v], z[4 * v + 1], z[4 * v + 2], z[4 * v + 3]);
            mbar_arrive_cluster(mapa_u32(smem_u32(&sh.recv_bar), dest));
          }
        }
        // the four warps that hold this block's own columns finish them
        if (ok && half == (int)(rank & 1u)) {
          bool got = mbar_try_wait_cluster(&sh.recv_bar, 0);
          if (!got) {
            const uint64_t t0 = global_timer_ns();
            while (!(got = mbar_try_wait_cluster(&sh.recv_bar, 0))) {
              if (*abortp) break;
              if (global_timer_ns() - t0 > wait_limit_ns(g.status)) {
                *abortp = 1;
                atomicCAS(g.status, 0, (int)ERR_EPILOGUE);
                break;
              }
            }
          }
          if (got) {
            // eight columns at a time in a loop that is not unrolled (see the note on the compact
            // tails below); partials added in ascending rank order, this block's own from TMEM
            const int cbase = (int)rank * 32;
#pragma unroll 1
            for (int s8 = 0; s8 < 32; s8 += 8) {
              uint32_t r8[8];
              tmem_ld_8cols(lane_addr + (uint32_t)(cbase + s8), r8);
              tmem_ld_wait();
              float z8[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) z8[j] = 0.f;
#pragma unroll 1
              for (int sp = 0; sp < g.splits; ++sp) {
                if (sp == (int)rank) {
#pragma unroll
                  for (int j = 0; j < 8; ++j) z8[j] += __uint_as_float(r8[j]);
                } else {
                  const float4* src =
                      reinterpret_cast<const float4*>(recv + ((size_t)sp * kBM + row) * 32 + s8);
                  const float4 t0 = src[0], t1 = src[1];
                  z8[0] += t0.x; z8[1] += t0.y; z8[2] += t0.z; z8[3] += t0.w;
                  z8[4] += t1.x; z8[5] += t1.y; z8[6] += t1.z; z8[7] += t1.w;
                }
              }
              uint32_t h4[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float a0 = z8[2 * j] + bias_pre, a1 = z8[2 * j + 1] + bias_pre;
                __nv_bfloat162 h2 = __floats2bfloat162_rn(a0 > 0.f ? a0 : 0.f, a1 > 0.f ? a1 : 0.f);
                h4[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              if (m_ok) {
                const int cc = cbase + s8;
                const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(h4);
                *reinterpret_cast<uint4*>(g.out_mb + ((size_t)p * g.M + m) * g.N + n0 + cc) =
                    make_uint4(h4[0], h4[1], h4[2], h4[3]);
                __nv_bfloat16* dbm = g.out_bm + ((size_t)p * g.N + n0 + cc) * g.M + m;
#pragma unroll
                for (int j = 0; j < 8; ++j) dbm[(size_t)j * g.M] = hh[j];
              }
            }
          }
        }
      }
      if (!CLUSTER && ALLOW_SPLIT && g.splits > 1) {   // the register-capped build is never used with a split
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
          sh.last_flag = last;
        }
        epilogue_barrier();
        finisher = sh.last_flag != 0;
      }
      if (finisher) {
        const float my_bias = EPI != EPI_DGRAD ? bias_pre : 0.f;
        float dsum = 0.f;
        float* lg = reinterpret_cast<float*>(smem);          // last layer: logits [N][M]
        // Hidden-layer forward and dgrad tails of an unsplit tile: eight columns at a time in a
        // loop that is NOT unrolled.  A tile's tail runs once per block, so its cost is largely
        // the fetch of its instructions; a short body that is reused beats a long one that is not.
        // Same values in the same order as the general path below.  The batch and the tile width
        // are multiples of 16, so a group of eight columns is inside the batch or outside it.
        const bool compact = EPI != EPI_FWD_LAST && (!ALLOW_SPLIT || g.splits == 1);
        if (compact) {
          const __nv_bfloat16* mrow = EPI == EPI_DGRAD
              ? g.mask_mb + ((size_t)p * g.M + m0 + row) * g.N + n0 : nullptr;
          uint4 mk8 = mk[0];                                  // first group, fetched before the wait
#pragma unroll 1
          for (int c0 = half * 32; c0 < g.BN; c0 += 64) {
#pragma unroll 1
            for (int s8 = 0; s8 < 32; s8 += 8) {
              const int cc = c0 + s8;
              if (cc >= g.BN) break;
              uint32_t r8[8];
              tmem_ld_8cols(lane_addr + (uint32_t)cc, r8);
              // mask of the next group of this warp, in flight while this one is finished
              uint4 mk8n = make_uint4(0, 0, 0, 0);
              if (EPI == EPI_DGRAD) {
                const int cn = s8 < 24 ? cc + 8 : c0 + 64;
                if (m_ok && cn < g.BN && n0 + cn < g.N)
                  mk8n = *reinterpret_cast<const uint4*>(mrow + cn);
              }
              tmem_ld_wait();
              const bool valid = n0 + cc < g.N;
              float z8[8];
              const __nv_bfloat16* mh = reinterpret_cast<const __nv_bfloat16*>(&mk8);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float v = __uint_as_float(r8[j]);
                if (EPI == EPI_DGRAD) {
                  v = (valid && __bfloat162float(mh[j]) > 0.f) ? v : 0.f;   // ReLU'(0) = 0
                  dsum += v;
                } else {
                  v += my_bias;
                  v = v > 0.f ? v : 0.f;
                }
                z8[j] = v;
              }
              uint32_t h4[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(z8[2 * j], z8[2 * j + 1]);
                h4[j] = *reinterpret_cast<uint32_t*>(&h2);
              }
              if (m_ok && valid) {
                const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(h4);
                *reinterpret_cast<uint4*>(g.out_mb + ((size_t)p * g.M + m) * g.N + n0 + cc) =
                    make_uint4(h4[0], h4[1], h4[2], h4[3]);
                __nv_bfloat16* dbm = g.out_bm + ((size_t)p * g.N + n0 + cc) * g.M + m;
#pragma unroll
                for (int j = 0; j < 8; ++j) dbm[(size_t)j * g.M] = hh[j];
              }
              mk8 = mk8n;
            }
          }
        }
        for (int c0 = compact ? g.BN : half * 32; c0 < g.BN; c0 += 64) {
          float z[32];
          int ncols;
          if (!ALLOW_SPLIT || g.splits == 1) {
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
          sh.colsum[half][row] = dsum;
          epilogue_barrier();
          if (half == 0 && m_ok) {
            float* ub = g.mom.u ? g.mom.u + (size_t)p * g.mom.u_stride + g.bias_off + m : nullptr;
            local_update(bias + m, bias_pre, ub, g.mom.read_u, sh.colsum[0][row] + sh.colsum[1][row],
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
            // the row's logits into registers first (at most 32 classes), so that no load waits
            // for arithmetic of an earlier class.  Exponentials and the logarithm are the hardware
            // approximations (relative error of a few 1e-7 for arguments of this size, far below
            // the bf16 rounding of dZ_L that follows).
            const float* zr = lg + t * C;
            float zv[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) zv[c] = c < C ? zr[c] : -INFINITY;
            float mx = zv[0];
#pragma unroll
            for (int c = 1; c < 32; ++c) mx = fmaxf(mx, zv[c]);
            float se = 0.f;
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (c < C) se += __expf(zv[c] - mx);                 // ascending c
            const float lse = mx + __logf(se);
            const int yb = label_pre;
            lossp[t] = lse - zr[yb];
            const float inv_b = 1.0f / (float)g.N;
            uint32_t packed[16];
#pragma unroll
            for (int c2 = 0; c2 < 16; ++c2) {
              float gr[2];
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const int c = 2 * c2 + h;
                gr[h] = 0.f;
                if (c < C) {
                  gr[h] = (__expf(zv[c] - lse) - (c == yb ? 1.f : 0.f)) * inv_b;
                  dzs[t * C + c] = gr[h];
                  g.dz_mb[((size_t)p * C + c) * g.N + t] = __float2bfloat16_rn(gr[h]);
                }
              }
              __nv_bfloat162 h2 = __floats2bfloat162_rn(gr[0], gr[1]);
              packed[c2] = *reinterpret_cast<uint32_t*>(&h2);
            }
            // the row of dZ_L [B, cpad] in 16-byte pieces (cpad is a multiple of 8; the padding
            // columns are written as zeros and never read)
            uint4* drow = reinterpret_cast<uint4*>(g.dz_bm + ((size_t)p * g.N + t) * g.cpad);
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (v * 8 < g.cpad)
                drow[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2],
                                     packed[4 * v + 3]);
          }
          epilogue_barrier();
          // loss: every warp adds its 32 rows, thread 0 the warps' sums; bias gradient of class c:
          // a warp adds the rows lane, lane + 32, ... and then its lanes, in a fixed order
          {
            float sl = t < g.N ? lossp[t] : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sl += __shfl_xor_sync(0xffffffffu, sl, o);
            if (lane == 0) sh.colsum[0][ew] = sl;
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
            for (int w = 0; w < nw; ++w) sl += sh.colsum[0][w];
            g.loss_out[(size_t)p * g.loss_stride] = sl / (float)g.N;
          }
        }
      }
    }
  }
}

}  // namespace gemm
}  // namespace mavg
