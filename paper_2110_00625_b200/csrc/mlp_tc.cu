// Tensor-core MLP learner step: the three matrix products of every layer run on tcgen05 with
// TMA-fed shared-memory operands and the accumulator in tensor memory.
//
// Every product is arranged so that the 128-row MMA dimension is a feature dimension and the
// batch (16..256 rows) is the MMA's N or K:
//   forward   Z^T[out, B]  = W[out, in]    . A[B, in]^T        contraction over in
//   dgrad     dA^T[in, B]  = W^T[in, out]  . dZ[B, out]^T      contraction over out
//   wgrad     dW[out, in]  = dZ^T[out, B]  . A^T[in, B]^T      contraction over the batch
// All operands are K-major bf16, so activations and dZ are kept in both orientations
// ([B, f] and [f, B]) and the weights' bf16 copy in both ([out, in] and, for layers >= 2,
// [in, out]); the producing epilogues write both.  fp32 master weights take the SGD step of
// Algorithm 1 in the wgrad epilogue, which also refreshes the bf16 copies.
// Forward and dgrad write fp32 partial tiles (split over the contraction when there are too few
// tiles to fill the GPU); small finishing kernels add the partials in a fixed order and apply
// bias/ReLU or the ReLU mask and the bias step.
#include <cuda.h>

#include <algorithm>

#include "mlp.cuh"
#include "tc_ptx.cuh"

namespace mavg {
namespace {

using namespace tc;

constexpr int kBM = 128;        // MMA M (rows of operand A per tile)
constexpr int kBK = 64;         // contraction elements per pipeline stage (128 bytes of bf16)
constexpr int kThreads = 320;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
constexpr int kStageBytes = 8 * 32 * 33 * 4;   // per-warp 32x32 fp32 turn-around tiles (wgrad)
constexpr int kMaxStages = 8;
constexpr int kATileBytes = kBM * kBK * 2;

enum { EPI_PARTIAL = 0, EPI_WGRAD_SGD = 1 };
enum { ERR_PRODUCER = 11, ERR_MMA = 12, ERR_EPILOGUE = 13 };

struct TcArgs {
  int M, N;                 // valid rows of A and of B
  int BN;                   // N tile: multiple of 16, <= 256
  int n_tiles, splits, kb_per_split, nkb, stages;
  int a_batched, b_batched; // 0: the operand is shared by all learners
  int P;
  uint32_t tmem_cols;
  // EPI_PARTIAL: part[((split*P + p)*N + n)*part_ld + m]
  float* part;
  int64_t part_ld;
  // EPI_WGRAD_SGD: A rows are output features o, B rows input features i
  float* rep;               // fp32 masters, W[o, i] at rep[p*rep_stride + w_off + o*in + i]
  int64_t rep_stride, w_off;
  int in, out;
  __nv_bfloat16* w16;       // bf16 copy [out, in] at w16[p*w16_stride + sh_off + o*in + i]
  int64_t w16_stride, sh_off;
  __nv_bfloat16* wt16;      // bf16 copy [in, out_pad] or null
  int64_t wt16_stride, sht_off;
  int out_pad;
  float gamma;
  int* status;
};

template <int EPI>
__global__ void __launch_bounds__(kThreads)
k_tc_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
          const TcArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

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
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int i = 0; i < count; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&empty_bar[s], (u & 1) ^ 1, abortp, g.status, ERR_PRODUCER)) break;
        uint8_t* sa = smem + (size_t)s * stage_bytes;
        mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
        tma_load_3d(sa, &tmA, &full_bar[s], (kb0 + i) * kBK, m0, g.a_batched ? p : 0);
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
      const uint32_t idesc = idesc_bf16_f32(kBM, g.BN);
      bool ok = true;
      for (int i = 0; i < count; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&full_bar[s], u & 1, abortp, g.status, ERR_MMA)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        const uint64_t adesc = smem_desc_k_sw128(sa);
        const uint64_t bdesc = smem_desc_k_sw128(sa + kATileBytes);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per MMA
          umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (uint32_t)((i | k) != 0));
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
    const bool ok = mbar_wait(&acc_bar, 0, abortp, g.status, ERR_EPILOGUE);
    tc_fence_after_sync();
    if (ok) {
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
      float* stage = reinterpret_cast<float*>(smem + (size_t)stages * stage_bytes) + ew * (32 * 33);
      for (int c0 = half * 32; c0 < g.BN; c0 += 64) {
        uint32_t r[32];
        if (c0 + 32 <= g.BN) {
          tmem_ld_32x32(lane_addr + (uint32_t)c0, r);
        } else {                             // BN is a multiple of 16
          uint32_t h[16];
          tmem_ld_16cols(lane_addr + (uint32_t)c0, h);
#pragma unroll
          for (int j = 0; j < 16; ++j) { r[j] = h[j]; r[16 + j] = 0u; }
        }
        tmem_ld_wait();
        const int ncols = min(32, g.BN - c0);
        if (EPI == EPI_PARTIAL) {
          const int m = m0 + row;
          if (m < g.M) {
            float* dst = g.part + ((size_t)(split * g.P + p) * g.N) * g.part_ld + m;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int n = n0 + c0 + j;
              if (j < ncols && n < g.N) dst[(size_t)n * g.part_ld] = __uint_as_float(r[j]);
            }
          }
        } else {
          // The accumulator arrives with one weight row per lane.  It is turned through shared
          // memory so that the lanes of a warp walk along a row: every access to the fp32 masters
          // and to the [out, in] bf16 copy is then a contiguous 128 / 64 bytes per row.
#pragma unroll
          for (int j = 0; j < 32; ++j) stage[lane * 33 + j] = __uint_as_float(r[j]);
          __syncwarp();
          const int o_base = m0 + q * 32;
          const int i = n0 + c0 + lane;
          const bool col_ok = lane < ncols && i < g.in;
          float* wcol = g.rep + (size_t)p * g.rep_stride + g.w_off + (size_t)o_base * g.in + i;
          __nv_bfloat16* hcol =
              g.w16 + (size_t)p * g.w16_stride + g.sh_off + (size_t)o_base * g.in + i;
          float wv[32];
#pragma unroll
          for (int rr = 0; rr < 32; ++rr)
            wv[rr] = (col_ok && o_base + rr < g.out) ? wcol[(size_t)rr * g.in] : 0.f;
#pragma unroll
          for (int rr = 0; rr < 32; ++rr) {
            const float w = fmaf(-g.gamma, stage[rr * 33 + lane], wv[rr]);
            if (col_ok && o_base + rr < g.out) {
              wcol[(size_t)rr * g.in] = w;
              hcol[(size_t)rr * g.in] = __float2bfloat16_rn(w);
            }
            stage[rr * 33 + lane] = w;
          }
          __syncwarp();
          if (g.wt16) {                       // [in, out] copy: lanes walk along out again
            const int o = o_base + lane;
            if (o < g.out) {
              __nv_bfloat16* tcol = g.wt16 + (size_t)p * g.wt16_stride + g.sht_off + o;
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const int ii = n0 + c0 + j;
                if (j < ncols && ii < g.in)
                  tcol[(size_t)ii * g.out_pad] = __float2bfloat16_rn(stage[lane * 33 + j]);
              }
            }
          }
          __syncwarp();
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, g.tmem_cols);
}

// ------------------------------------------------------------------------------ finishing kernels
// Forward: z = sum_s part_s + bias;  hidden layers store relu(z) as bf16 in both orientations,
// the last layer stores fp32 logits.  grid (ceil(out/32), ceil(B/32), P), block (32, 8).
template <bool LAST>
__global__ void __launch_bounds__(256)
k_fwd_finish(const float* __restrict__ part, int S, int P, int B, int out,
             const float* __restrict__ rep, int64_t rep_stride, int64_t b_off,
             __nv_bfloat16* __restrict__ act, __nv_bfloat16* __restrict__ act_t,
             float* __restrict__ logits) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int p = blockIdx.z, o0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int o = o0 + tx;
  const float bias = o < out ? rep[(size_t)p * rep_stride + b_off + o] : 0.f;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int b = b0 + ty + 8 * r;
    if (o < out && b < B) {
      float z = 0.f;
      for (int s = 0; s < S; ++s) z += part[((size_t)(s * P + p) * B + b) * out + o];
      z += bias;
      if (LAST) {
        logits[((size_t)p * B + b) * out + o] = z;
      } else {
        __nv_bfloat16 a = __float2bfloat16_rn(z > 0.f ? z : 0.f);
        act[((size_t)p * B + b) * out + o] = a;
        tile[ty + 8 * r][tx] = a;
      }
    }
  }
  if (!LAST) {
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int oo = o0 + ty + 8 * r, b = b0 + tx;
      if (oo < out && b < B) act_t[((size_t)p * out + oo) * B + b] = tile[tx][ty + 8 * r];
    }
  }
}

// dgrad: dA = sum_s part_s;  dZ = dA where the forward activation was positive, else 0
// (ReLU'(0) = 0); stores dZ as bf16 in both orientations and takes the bias step of the layer
// that produced the activation:  b[f] -= gamma * sum_b dZ[b, f]  (unrounded dZ, fixed order).
// grid (ceil(feat/32), P), block (32, 8).
__global__ void __launch_bounds__(256)
k_dgrad_finish(const float* __restrict__ part, int S, int P, int B, int feat,
               const __nv_bfloat16* __restrict__ act, __nv_bfloat16* __restrict__ dz,
               __nv_bfloat16* __restrict__ dz_t, float* __restrict__ rep, int64_t rep_stride,
               int64_t b_off, float gamma) {
  __shared__ __nv_bfloat16 tile[32][33];
  __shared__ float red[8][32];
  const int p = blockIdx.y, f0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int f = f0 + tx;
  float acc = 0.f;
  for (int bc = 0; bc < B; bc += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int b = bc + ty + 8 * r;
      __nv_bfloat16 q = __float2bfloat16_rn(0.f);
      if (f < feat && b < B) {
        float d = 0.f;
        for (int s = 0; s < S; ++s) d += part[((size_t)(s * P + p) * B + b) * feat + f];
        const size_t at = ((size_t)p * B + b) * feat + f;
        d = __bfloat162float(act[at]) > 0.f ? d : 0.f;
        acc += d;
        q = __float2bfloat16_rn(d);
        dz[at] = q;
      }
      tile[ty + 8 * r][tx] = q;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int ff = f0 + ty + 8 * r, b = bc + tx;
      if (ff < feat && b < B) dz_t[((size_t)p * feat + ff) * B + b] = tile[tx][ty + 8 * r];
    }
    __syncthreads();
  }
  red[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && f < feat) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) s += red[r][tx];
    float* bias = rep + (size_t)p * rep_stride + b_off;
    bias[f] = fmaf(-gamma, s, bias[f]);
  }
}

// bf16 copies of the global model w~ (shared by all learners at the first step of a round, when
// every replica equals w~).  One launch per layer; grid-stride over the layer's weights.
__global__ void __launch_bounds__(256)
k_shadow_from_global(const float* __restrict__ w, int64_t w_off, int in, int out,
                     __nv_bfloat16* __restrict__ w16, int64_t sh_off,
                     __nv_bfloat16* __restrict__ wt16, int64_t sht_off, int out_pad) {
  const int64_t total = (int64_t)in * out;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    __nv_bfloat16 h = __float2bfloat16_rn(w[w_off + t]);
    w16[sh_off + t] = h;
    if (wt16) {
      const int o = (int)(t / in), i = (int)(t % in);
      wt16[sht_off + (int64_t)i * out_pad + o] = h;
    }
  }
}

// ---------------------------------------------------------------------------------- host side
size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct TcLayout {
  int L;
  int cpad;                                  // last layer's dZ row length (multiple of 8)
  int64_t n16, nt16;                         // elements per bf16 copy row
  int64_t sh_off[MAVG_MAX_LAYERS], sht_off[MAVG_MAX_LAYERS];
  int out_pad[MAVG_MAX_LAYERS];
  size_t xg, xt;
  size_t act[MAVG_MAX_LAYERS + 1], act_t[MAVG_MAX_LAYERS + 1];
  size_t dz[MAVG_MAX_LAYERS + 1], dz_t[MAVG_MAX_LAYERS + 1];
  size_t logits, dz_last;
  size_t part, part_bytes;
  size_t w16, wt16, w16g, wt16g;
  size_t end;
};

struct GemmPlan { int m_tiles, n_tiles, splits, kb_per_split, nkb, BN, stages; uint32_t tmem_cols; };

GemmPlan plan_partial(int M, int N, int K, int P, int sm_count) {
  GemmPlan g{};
  g.BN = (N + 15) / 16 * 16;
  g.m_tiles = (M + kBM - 1) / kBM;
  g.n_tiles = 1;
  g.nkb = (K + kBK - 1) / kBK;
  int tiles = g.m_tiles * P;
  int want = tiles >= sm_count ? 1 : (sm_count + tiles - 1) / tiles;
  if (want > g.nkb) want = g.nkb;
  g.kb_per_split = (g.nkb + want - 1) / want;
  g.splits = (g.nkb + g.kb_per_split - 1) / g.kb_per_split;
  int stage_bytes = kATileBytes + g.BN * kBK * 2;
  g.stages = 200 * 1024 / stage_bytes;
  if (g.stages > kMaxStages) g.stages = kMaxStages;
  if (g.stages > g.kb_per_split) g.stages = g.kb_per_split < 2 ? 2 : g.kb_per_split;
  g.tmem_cols = 32;
  while ((int)g.tmem_cols < g.BN) g.tmem_cols <<= 1;
  return g;
}

GemmPlan plan_wgrad(int out, int in, int B) {
  GemmPlan g{};
  g.BN = in >= 128 ? 128 : (in + 15) / 16 * 16;
  g.m_tiles = (out + kBM - 1) / kBM;
  g.n_tiles = (in + g.BN - 1) / g.BN;
  g.nkb = (B + kBK - 1) / kBK;
  g.splits = 1;
  g.kb_per_split = g.nkb;
  g.stages = g.nkb < 2 ? 2 : (g.nkb > 4 ? 4 : g.nkb);
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
  int64_t o16 = 0, ot16 = 0;
  for (int l = 0; l < L; ++l) {
    const int in = cfg->dims[l], out = cfg->dims[l + 1];
    t.sh_off[l] = o16;
    o16 += (int64_t)up((size_t)in * out, 64);
    t.out_pad[l] = (out + 7) / 8 * 8;
    t.sht_off[l] = ot16;
    if (l > 0) ot16 += (int64_t)up((size_t)in * t.out_pad[l], 64);
  }
  t.n16 = o16;
  t.nt16 = ot16 > 0 ? ot16 : 64;
  size_t off = up(base, 1024);
  auto take = [&](size_t bytes) { size_t r = off; off = up(off + bytes, 1024); return r; };
  t.xg = take(rows * cfg->dims[0] * 2);
  t.xt = take(rows * cfg->dims[0] * 2);
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
  }
  t.logits = take(rows * cfg->dims[L] * 4);
  t.dz_last = take(rows * cfg->dims[L] * 4);
  size_t pb = 0;
  for (int l = 1; l <= L; ++l) {
    GemmPlan f = plan_partial(cfg->dims[l], B, cfg->dims[l - 1], P, sm_count);
    pb = std::max(pb, (size_t)f.splits * rows * cfg->dims[l] * 4);
    if (l > 1) {
      GemmPlan d = plan_partial(cfg->dims[l - 1], B, cfg->dims[l], P, sm_count);
      pb = std::max(pb, (size_t)d.splits * rows * cfg->dims[l - 1] * 4);
    }
  }
  t.part_bytes = pb;
  t.part = take(pb);
  t.w16 = take((size_t)P * t.n16 * 2);
  t.wt16 = take((size_t)P * t.nt16 * 2);
  t.w16g = take((size_t)t.n16 * 2);
  t.wt16g = take((size_t)t.nt16 * 2);
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
  CUtensorMap wt[MAVG_MAX_LAYERS + 1], wtg[MAVG_MAX_LAYERS + 1];     // [in, out] copies (l >= 2)
  CUtensorMap act_in[MAVG_MAX_LAYERS + 1];    // [B, d_{l-1}] input activations of layer l
  CUtensorMap act_in_t[MAVG_MAX_LAYERS + 1];  // [d_{l-1}, B]
  CUtensorMap dz[MAVG_MAX_LAYERS + 1];        // [B, d_l]
  CUtensorMap dz_t[MAVG_MAX_LAYERS + 1];      // [d_l, B]
  GemmPlan fwd[MAVG_MAX_LAYERS + 1], dgrad[MAVG_MAX_LAYERS + 1], wgrad[MAVG_MAX_LAYERS + 1];
};

// bf16 tensor [batch, rows, inner] with the given strides (in elements); box = 64 x box_rows.
bool encode_map(TcState* st, CUtensorMap* m, void* ptr, int inner, int rows, int batch,
                int64_t row_stride, int64_t batch_stride, int box_rows, std::string* why) {
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)row_stride * 2, (cuuint64_t)batch_stride * 2};
  cuuint32_t box[3] = {(cuuint32_t)kBK, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r = st->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptr, dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    if (why) *why = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
    return false;
  }
  return true;
}

template <int EPI>
cudaError_t launch_gemm(mavg_ctx* c, int cls, const CUtensorMap& a, const CUtensorMap& b,
                        const GemmPlan& pl, TcArgs g) {
  g.BN = pl.BN;
  g.n_tiles = pl.n_tiles;
  g.splits = pl.splits;
  g.kb_per_split = pl.kb_per_split;
  g.nkb = pl.nkb;
  g.stages = pl.stages;
  g.tmem_cols = pl.tmem_cols;
  g.P = c->cfg.P;
  g.status = (int*)ws_ptr(c, c->ws.status);
  const size_t smem = (size_t)pl.stages * (kATileBytes + pl.BN * kBK * 2) + 1024 +
                      (EPI == EPI_WGRAD_SGD ? kStageBytes : 0);
  dim3 grid((unsigned)(pl.m_tiles * pl.n_tiles * pl.splits), (unsigned)c->cfg.P);
  prof_begin(c, cls);
  k_tc_gemm<EPI><<<grid, kThreads, smem, c->stream>>>(a, b, g);
  prof_end(c);
  return cudaGetLastError();
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
    st->fwd[l] = plan_partial(out, B, in, P, kPlanSmCount);
    st->wgrad[l] = plan_wgrad(out, in, B);
    __nv_bfloat16* w16 = (__nv_bfloat16*)bf(t.w16) + t.sh_off[l - 1];
    __nv_bfloat16* w16g = (__nv_bfloat16*)bf(t.w16g) + t.sh_off[l - 1];
    ok = ok && encode_map(st, &st->w[l], w16, in, out, P, in, t.n16, kBM, &why);
    ok = ok && encode_map(st, &st->wg[l], w16g, in, out, 1, in, t.n16, kBM, &why);
    void* a_in = l == 1 ? bf(t.xg) : bf(t.act[l - 1]);
    void* a_in_t = l == 1 ? bf(t.xt) : bf(t.act_t[l - 1]);
    ok = ok && encode_map(st, &st->act_in[l], a_in, in, B, P, in, (int64_t)B * in,
                          st->fwd[l].BN, &why);
    ok = ok && encode_map(st, &st->act_in_t[l], a_in_t, B, in, P, B, (int64_t)B * in,
                          st->wgrad[l].BN, &why);
    ok = ok && encode_map(st, &st->dz_t[l], bf(t.dz_t[l]), B, out, P, B, (int64_t)B * out, kBM,
                          &why);
    if (l > 1) {
      st->dgrad[l] = plan_partial(in, B, out, P, kPlanSmCount);
      __nv_bfloat16* wt16 = (__nv_bfloat16*)bf(t.wt16) + t.sht_off[l - 1];
      __nv_bfloat16* wt16g = (__nv_bfloat16*)bf(t.wt16g) + t.sht_off[l - 1];
      ok = ok && encode_map(st, &st->wt[l], wt16, out, in, P, t.out_pad[l - 1], t.nt16, kBM, &why);
      ok = ok && encode_map(st, &st->wtg[l], wt16g, out, in, 1, t.out_pad[l - 1], t.nt16, kBM, &why);
      ok = ok && encode_map(st, &st->dz[l], bf(t.dz[l]), out, B, P, dz_ld, (int64_t)B * dz_ld,
                            st->dgrad[l].BN, &why);
    }
  }
  if (!ok) {
    c->err = why;
    return MAVG_ERR_CUDA;
  }
  // 227 KB per block in all, of which a few hundred bytes are the kernel's static barriers
  constexpr int kMaxDynSmem = 226 * 1024;
  e = cudaFuncSetAttribute(k_tc_gemm<EPI_PARTIAL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kMaxDynSmem);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_tc_gemm<EPI_WGRAD_SGD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kMaxDynSmem);
  if (e != cudaSuccess) {
    c->err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
    cudaGetLastError();   // reported here; do not leave it pending for a later call
    return MAVG_ERR_CUDA;
  }
  return MAVG_OK;
}

void tc_teardown(mavg_ctx* c) {
  delete (TcState*)c->mlp;
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
    k_shadow_from_global<<<grid, 256, 0, c->stream>>>(
        c->buf.global_w, ly.w_off, ly.in, ly.out, (__nv_bfloat16*)(ws + t.w16g), t.sh_off[l - 1],
        l > 1 ? (__nv_bfloat16*)(ws + t.wt16g) : nullptr, t.sht_off[l - 1], t.out_pad[l - 1]);
    prof_end(c);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t tc_step(mavg_ctx* c, int64_t round, int step) {
  TcState* st = (TcState*)c->mlp;
  const TcLayout& t = st->lay;
  const mavg_config& cfg = c->cfg;
  const int P = cfg.P, B = cfg.B, L = cfg.n_layers;
  char* ws = (char*)c->buf.workspace;
  auto bfp = [&](size_t off) { return (__nv_bfloat16*)(ws + off); };
  int32_t* idx = (int32_t*)ws_ptr(c, c->ws.idx);
  int32_t* labels = (int32_t*)ws_ptr(c, c->ws.labels);
  float* losses = (float*)ws_ptr(c, c->ws.losses);
  float* part = (float*)(ws + t.part);
  float* logits = (float*)(ws + t.logits);
  float* dz_last = (float*)(ws + t.dz_last);
  const bool shared_w = c->replicas_equal_global;   // first step after a (re-)broadcast
  cudaError_t e;
  if ((e = launch_batch_indices(c, round, step, 0, P, idx, labels)) != cudaSuccess) return e;
  if ((e = launch_gather(c, idx, 1, nullptr, bfp(t.xg), bfp(t.xt))) != cudaSuccess) return e;

  for (int l = 1; l <= L; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    TcArgs g{};
    g.M = ly.out; g.N = B;
    g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
    g.part = part; g.part_ld = ly.out;
    if ((e = launch_gemm<EPI_PARTIAL>(c, MAVG_K_FWD, shared_w ? st->wg[l] : st->w[l],
                                      st->act_in[l], st->fwd[l], g)) != cudaSuccess)
      return e;
    dim3 grid((ly.out + 31) / 32, (B + 31) / 32, P), block(32, 8);
    prof_begin(c, MAVG_K_FWD);
    if (l < L)
      k_fwd_finish<false><<<grid, block, 0, c->stream>>>(part, st->fwd[l].splits, P, B, ly.out,
                                                         c->buf.replicas, c->buf.replica_stride,
                                                         ly.b_off, bfp(t.act[l]), bfp(t.act_t[l]),
                                                         nullptr);
    else
      k_fwd_finish<true><<<grid, block, 0, c->stream>>>(part, st->fwd[l].splits, P, B, ly.out,
                                                        c->buf.replicas, c->buf.replica_stride,
                                                        ly.b_off, nullptr, nullptr, logits);
    prof_end(c);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  const int C = cfg.dims[L];
  if ((e = launch_softmax_ce(c, logits, C, labels, losses + (step - 1), cfg.K, dz_last, C,
                             bfp(t.dz[L]), t.cpad, bfp(t.dz_t[L]), B, true)) != cudaSuccess)
    return e;

  for (int l = L; l >= 1; --l) {
    const MlpLayer& ly = c->layers[l - 1];
    if (l > 1) {
      const MlpLayer& below = c->layers[l - 2];
      TcArgs g{};
      g.M = ly.in; g.N = B;
      g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
      g.part = part; g.part_ld = ly.in;
      if ((e = launch_gemm<EPI_PARTIAL>(c, MAVG_K_DGRAD, shared_w ? st->wtg[l] : st->wt[l],
                                        st->dz[l], st->dgrad[l], g)) != cudaSuccess)
        return e;
      dim3 grid((ly.in + 31) / 32, P), block(32, 8);
      prof_begin(c, MAVG_K_DGRAD);
      k_dgrad_finish<<<grid, block, 0, c->stream>>>(part, st->dgrad[l].splits, P, B, ly.in,
                                                    bfp(t.act[l - 1]), bfp(t.dz[l - 1]),
                                                    bfp(t.dz_t[l - 1]), c->buf.replicas,
                                                    c->buf.replica_stride, below.b_off,
                                                    cfg.local_lr);
      prof_end(c);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    TcArgs g{};
    g.M = ly.out; g.N = ly.in;
    g.a_batched = 1; g.b_batched = 1;
    g.rep = c->buf.replicas; g.rep_stride = c->buf.replica_stride; g.w_off = ly.w_off;
    g.in = ly.in; g.out = ly.out;
    g.w16 = bfp(t.w16); g.w16_stride = t.n16; g.sh_off = t.sh_off[l - 1];
    g.wt16 = l > 1 ? bfp(t.wt16) : nullptr; g.wt16_stride = t.nt16; g.sht_off = t.sht_off[l - 1];
    g.out_pad = t.out_pad[l - 1];
    g.gamma = cfg.local_lr;
    if ((e = launch_gemm<EPI_WGRAD_SGD>(c, MAVG_K_WGRAD_SGD, st->dz_t[l], st->act_in_t[l],
                                        st->wgrad[l], g)) != cudaSuccess)
      return e;
  }
  return cudaSuccess;
}

}  // namespace mavg
