// All K local steps of a round (the inner loop of Algorithm 1 for every learner) in ONE persistent
// kernel, for workloads whose single products are too small to fill the GPU or to pay for a
// launch each.  One block per SM; every block walks the same list of work units and runs the
// units that fall to it.  The units are the tiles of the per-launch kernels -- a forward or dgrad
// output tile with its fused tail (gemm_unit.cuh), a run of weight-gradient + SGD tiles
// (wgrad_unit.cuh), a slice of the minibatch gather -- so the arithmetic, and with it every bit of
// the result, is that of the launch-by-launch schedule of mlp_tc.cu.
//
// What a launch boundary used to order is ordered per learner by counters in global memory: a
// unit that finishes adds one to the counter of its (kind, layer, learner); a unit that starts
// waits until the counters of what it reads (and of the readers of what it overwrites) have
// reached the value they must have at this step.  Units of one step are grouped; a group only
// depends on earlier groups, every block goes through the groups in the same order, and all
// blocks are resident at once (cooperative launch), so some block can always make progress.
// Groups of local step k (L layers; D_l = dgrad through layer l, WG_l = weight gradient + SGD of
// layer l, G = gather of a step's minibatch into the buffer of that step's parity):
//   [G(1) before the first step]  {F_1} ... {F_{L-1}}  {F_L + loss, G(k+1)}  {D_L}
//   {D_{L-1}, WG_L} ... {D_2, WG_3}  {WG_2, WG_1}
// so that the narrow groups (few tiles) run beside independent work.
// Every wait is bounded; a wait that runs out sets the status word, which makes every other wait
// of the launch give up as well.
#include <cuda.h>

#include <algorithm>

#include "gemm_unit.cuh"
#include "mlp.cuh"
#include "tc_state.cuh"
#include "wgrad_unit.cuh"

namespace mavg {
namespace {

using namespace tc;

constexpr int kRoundMaxLayers = 5;
constexpr int kRoundThreads = 352;     // warp 0 producer, 1 MMA issuer, 2-9 epilogue, 10 stores
constexpr int kGatherCols = 256;       // input columns per gather unit
enum { CNT_G = 0, CNT_F = 1, CNT_D = 2, CNT_WG = 3, CNT_KINDS = 4 };
enum { ERR_ROUND_DEP = 31 };

struct RoundLayer {
  int in, out;
  int64_t w_off, b_off;
  int f_BN, f_m_tiles, f_n_tiles, f_nkb;                 // forward plan
  int d_BN, d_m_tiles, d_nkb;                            // dgrad plan (l >= 2; rows = in)
  int w_nkb, w_m_tiles, w_n_tiles, w_chunk, w_n_chunks;  // weight-gradient plan
  __nv_bfloat16 *act, *act_t;                            // relu(z_l) [P,B,out] and [P,out,B] (l < L)
  __nv_bfloat16 *dz, *dz_t;                              // dZ_l [P,B,out or cpad] and [P,out,B]
};

struct RoundParams {
  // index l = 1..L as in TcState
  CUtensorMap w[kRoundMaxLayers + 1], wg[kRoundMaxLayers + 1];
  CUtensorMap w_mn[kRoundMaxLayers + 1], wg_mn[kRoundMaxLayers + 1];
  CUtensorMap act_in[kRoundMaxLayers + 1], act_in_t[kRoundMaxLayers + 1];
  CUtensorMap dz[kRoundMaxLayers + 1], dz_t[kRoundMaxLayers + 1];
  CUtensorMap w32[kRoundMaxLayers + 1], w32g[kRoundMaxLayers + 1], w16_st[kRoundMaxLayers + 1];
  CUtensorMap x_in[2], x_in_t[2];
  RoundLayer ly[kRoundMaxLayers + 1];
  int L, P, B, K, cpad;
  int first_shared;           // 1: every learner starts the round from w~ (step 1 reads w~)
  int stages;                 // pipeline depth of every forward / dgrad tile of this launch
  int w_slots, w_a_bufs, w_on_b;   // ring geometry of every weight-gradient run
  int g_slot_groups, g_col_splits;
  int64_t round;
  uint64_t seed;
  int64_t S;
  const void* x;
  int x_bf16;
  const int32_t* y;
  __nv_bfloat16* xg[2];
  __nv_bfloat16* xt[2];
  int32_t* labels[2];
  float* losses;
  float* replicas;
  const float* global_w;
  int64_t rep_stride;
  float gamma;
  int keep_w32;          // master tiles carry the L2 keep hint (see WgradArgs)
  int* counters;              // [CNT_KINDS][kRoundMaxLayers + 1][P], zero at launch
  int* status;
};

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Orders this thread's earlier generic-proxy accesses to global memory with later async-proxy
// (TMA) accesses, and the other way round.
__device__ __forceinline__ void fence_proxy_async_all() {
  asm volatile("fence.proxy.async;" ::: "memory");
}

__device__ __forceinline__ int* counter(const RoundParams& rp, int kind, int l, int p) {
  return rp.counters + ((size_t)(kind * (kRoundMaxLayers + 1) + l) * rp.P + p);
}

// Waits until *ctr >= target.  False if the wait was abandoned (time limit, or another wait of
// the launch gave up before).
__device__ __forceinline__ bool wait_count(const int* ctr, int target, int* status) {
  if (target <= 0) return true;
  if (ld_acquire(ctr) >= target) return true;
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (ld_acquire(ctr) < target) {
    if ((++spins & 0x3F) == 0) {
      if (*(volatile int*)status != 0) return false;
      if (global_timer_ns() - t0 > wait_limit_ns(status)) {
        atomicCAS(status, 0, (int)ERR_ROUND_DEP);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void signal_done(int* ctr) {
  __threadfence();
  atomicAdd(ctr, 1);
}

// Per-learner unit counts of one step, from the plans.
__device__ __forceinline__ int f_tiles(const RoundLayer& y) { return y.f_m_tiles * y.f_n_tiles; }
__device__ __forceinline__ int wg_items(const RoundLayer& y) { return y.w_m_tiles * y.w_n_chunks; }
__device__ __forceinline__ int g_units(const RoundParams& rp) { return rp.g_slot_groups * rp.g_col_splits; }

// ---- what each unit waits for (learner p, local step k) ------------------------------------------
// dZ_l of step k is complete for learner p
__device__ __forceinline__ bool dz_ready(const RoundParams& rp, int l, int p, int k) {
  if (l == rp.L) return wait_count(counter(rp, CNT_F, l, p), k, rp.status);
  return wait_count(counter(rp, CNT_D, l + 1, p), k * rp.ly[l + 1].d_m_tiles, rp.status);
}
__device__ __forceinline__ bool fwd_deps(const RoundParams& rp, int l, int p, int k) {
  bool ok;
  // input activations of this step
  if (l == 1) ok = wait_count(counter(rp, CNT_G, 0, p), k * g_units(rp), rp.status);
  else ok = wait_count(counter(rp, CNT_F, l - 1, p), k * f_tiles(rp.ly[l - 1]), rp.status);
  // W_l (bf16) as the previous step left it
  ok = ok && wait_count(counter(rp, CNT_WG, l, p), (k - 1) * wg_items(rp.ly[l]), rp.status);
  // the output A_l is still read (transposed) by the previous step's WG_{l+1}
  if (l < rp.L)
    ok = ok && wait_count(counter(rp, CNT_WG, l + 1, p), (k - 1) * wg_items(rp.ly[l + 1]), rp.status);
  return ok;
}
__device__ __forceinline__ bool dgrad_deps(const RoundParams& rp, int l, int p, int k) {
  return dz_ready(rp, l, p, k);
}
__device__ __forceinline__ bool gather_deps(const RoundParams& rp, int p, int k) {
  // the buffers of parity k & 1 were last read by WG_1 of step k - 2; and the gather counter of
  // a learner must reach k - 1 full steps before units of step k add to it (nothing else orders
  // the gathers of successive steps, and readers wait for "k steps' worth" of units)
  return wait_count(counter(rp, CNT_WG, 1, p), (k - 2) * wg_items(rp.ly[1]), rp.status) &&
         wait_count(counter(rp, CNT_G, 0, p), (k - 1) * g_units(rp), rp.status);
}

struct WgDeps {
  static constexpr bool kSignals = true;
  const RoundParams* rp;
  int l, k;
  __device__ __forceinline__ bool inputs_ready(int p, volatile int* abort_flag) const {
    bool ok = dz_ready(*rp, l, p, k);
    // dgrad through this layer still reads the bf16 weights this run overwrites
    if (ok && l >= 2) ok = wait_count(counter(*rp, CNT_D, l, p), k * rp->ly[l].d_m_tiles, rp->status);
    if (!ok) {
      *abort_flag = 1;
      return false;
    }
    fence_proxy_async_all();
    return true;
  }
  // called once the item's bulk stores have completed (their writes are then performed; the
  // release below publishes them)
  __device__ __forceinline__ void item_done(int p) const {
    signal_done(counter(*rp, CNT_WG, l, p));
  }
};

struct RoundShared {
  gemm::GemmShared g;
  wgrad::WgradShared w;
  int stop;                    // set when a unit was abandoned: every thread leaves the kernel
};
// staging of a gather unit, at the start of the (then idle) pipeline buffer
constexpr int kGatherPitch = kGatherCols + 8;      // bf16 elements per staged row (16-byte aligned)
struct GatherStage {
  int32_t sidx[32];
  __align__(16) __nv_bfloat16 tile[32][kGatherPitch];
};

// Eight consecutive elements of a dataset row as bf16 (round to nearest even).
__device__ __forceinline__ uint4 load8_bf16(const __nv_bfloat16* src) {
  return *reinterpret_cast<const uint4*>(src);
}
__device__ __forceinline__ uint4 load8_bf16(const float* src) {
  const float4 a = *reinterpret_cast<const float4*>(src);
  const float4 b = *reinterpret_cast<const float4*>(src + 4);
  __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
  __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
  return make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                    *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
}

// Threads 0..255: 32 batch slots of learner p, input columns [c_lo, c_hi) (at most kGatherCols,
// a multiple of 8).  Draws the slots' sample indices ("randomly sample a mini-batch",
// Algorithm 1), copies the rows as bf16 [P, B, d] and, through a shared-memory tile, their
// transpose [P, d, B].  All loads of a thread are issued before their first use.
template <typename TIN>
__device__ __forceinline__ void gather_slice(const RoundParams& rp, GatherStage& sh, int k, int p,
                                             int s0, int c_lo, int c_hi, bool write_labels) {
  const int tid = threadIdx.x;
  if (tid >= 256) return;
  const int B = rp.B, d = rp.ly[1].in;
  const TIN* x = reinterpret_cast<const TIN*>(rp.x);
  __nv_bfloat16* out_bf = rp.xg[k & 1];
  __nv_bfloat16* out_bft = rp.xt[k & 1];
  if (tid < 32) {
    const int s = s0 + tid;
    int32_t i = 0;
    if (s < B) {
      i = sample_index(rp.seed, rp.round, p, k, s, rp.P, rp.S);
      if (write_labels) rp.labels[k & 1][p * B + s] = rp.y[i];
    }
    sh.sidx[tid] = i;
  }
  asm volatile("bar.sync 2, 256;" ::: "memory");
  constexpr int kChunks = kGatherCols / 8;           // 16-byte chunks per staged row
  constexpr int kPerThread = 32 * kChunks / 256;
  uint4 v[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int q = tid + 256 * i;
    const int r = q / kChunks, c = c_lo + (q % kChunks) * 8;
    v[i] = make_uint4(0u, 0u, 0u, 0u);
    if (s0 + r < B && c < c_hi) v[i] = load8_bf16(x + (size_t)sh.sidx[r] * d + c);
  }
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int q = tid + 256 * i;
    const int r = q / kChunks, c8 = (q % kChunks) * 8, c = c_lo + c8;
    if (s0 + r < B && c < c_hi)
      *reinterpret_cast<uint4*>(out_bf + ((size_t)p * B + s0 + r) * d + c) = v[i];
    *reinterpret_cast<uint4*>(&sh.tile[r][c8]) = v[i];
  }
  asm volatile("bar.sync 2, 256;" ::: "memory");
  // transpose: a task is one column and eight consecutive slots (16 bytes of [P, d, B])
  for (int task = tid; task < kGatherCols * 4; task += 256) {
    const int so = task & 3, cl = task >> 2;
    const int c = c_lo + cl, s = s0 + so * 8;
    if (c < c_hi && s < B) {                         // B is a multiple of 16: all eight or none
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint16_t lo = *reinterpret_cast<const uint16_t*>(&sh.tile[so * 8 + 2 * j][cl]);
        const uint16_t hi = *reinterpret_cast<const uint16_t*>(&sh.tile[so * 8 + 2 * j + 1][cl]);
        w[j] = (uint32_t)lo | ((uint32_t)hi << 16);
      }
      *reinterpret_cast<uint4*>(out_bft + ((size_t)p * d + c) * B + s) =
          make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

__global__ void __launch_bounds__(kRoundThreads, 1)
k_mlp_round(const __grid_constant__ RoundParams rp) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) RoundShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5;
  const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
  const int L = rp.L, P = rp.P, K = rp.K;

  if (threadIdx.x == 0) {
    gemm::gemm_init_barriers(sh.g, rp.stages);
    wgrad::wgrad_init_barriers(sh.w, rp.w_slots);
    sh.g.abort_flag = 0;
    sh.w.abort_flag = 0;
    sh.stop = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&sh.g.tmem_slot, 256);      // widest accumulator: 128 lanes x 256 columns
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh.g.tmem_slot;

  // Phase bookkeeping of the barriers, identical in every thread of the block.
  uint32_t g_slabs = 0, g_tiles = 0;       // pipeline slabs / tiles of the GEMM units so far
  uint32_t w_tiles = 0, w_items = 0;       // tiles / items of the weight-gradient runs so far
  int rot = 0;                             // unit i of a segment runs on block (rot + i) % grid
  bool stop = false;

  // ---- one forward / dgrad tile ------------------------------------------------------------------
  // kind: EPI_FWD_HIDDEN, EPI_FWD_LAST, EPI_DGRAD; t: tile index inside the layer's launch
  auto gemm_unit = [&](int kind, int l, int k, int t) {
    const RoundLayer& y = rp.ly[l];
    const bool shared_w = rp.first_shared && k == 1;
    gemm::TcArgs g{};
    int per_p, p, bx;
    const CUtensorMap *ta, *tb;
    if (kind == gemm::EPI_DGRAD) {
      per_p = y.d_m_tiles;
      p = t / per_p; bx = t % per_p;
      g.M = y.in; g.N = rp.B; g.BN = y.d_BN; g.m_tiles = y.d_m_tiles; g.n_tiles = 1; g.nkb = y.d_nkb;
      g.bias_off = rp.ly[l - 1].b_off;
      g.out_bm = rp.ly[l - 1].dz; g.out_mb = rp.ly[l - 1].dz_t; g.mask_mb = rp.ly[l - 1].act_t;
      g.a_mn = 1;
      ta = shared_w ? &rp.wg_mn[l] : &rp.w_mn[l];
      tb = &rp.dz[l];
    } else {
      per_p = f_tiles(y);
      p = t / per_p; bx = t % per_p;
      g.M = y.out; g.N = rp.B; g.BN = y.f_BN; g.m_tiles = y.f_m_tiles; g.n_tiles = y.f_n_tiles;
      g.nkb = y.f_nkb;
      g.bias_off = y.b_off;
      if (kind == gemm::EPI_FWD_HIDDEN) {
        g.out_bm = y.act; g.out_mb = y.act_t;
      } else {
        g.labels = rp.labels[k & 1]; g.loss_out = rp.losses + (k - 1); g.loss_stride = K;
        g.dz_bm = y.dz; g.cpad = rp.cpad; g.dz_mb = y.dz_t;
      }
      ta = shared_w ? &rp.wg[l] : &rp.w[l];
      tb = l == 1 ? &rp.x_in[k & 1] : &rp.act_in[l];
    }
    g.splits = 1; g.kb_per_split = g.nkb; g.stages = rp.stages;
    g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
    g.P = P;
    g.bias_rep = rp.replicas;
    g.bias_in = shared_w ? rp.global_w : rp.replicas;
    g.bias_in_stride = shared_w ? 0 : rp.rep_stride;
    g.rep_stride = rp.rep_stride;
    g.gamma = rp.gamma;
    g.status = rp.status;
    if (threadIdx.x == 0) {
      const bool ok = kind == gemm::EPI_DGRAD ? dgrad_deps(rp, l, p, k) : fwd_deps(rp, l, p, k);
      if (!ok) sh.g.abort_flag = 1;
      fence_proxy_async_all();
    }
    __syncthreads();
    tc_fence_after_sync();
    if (!sh.g.abort_flag) {
      if (kind == gemm::EPI_FWD_HIDDEN)
        gemm::gemm_tile<gemm::EPI_FWD_HIDDEN, false>(*ta, *tb, g, bx, p, smem, sh.g, tmem_base, g_slabs, g_tiles);
      else if (kind == gemm::EPI_FWD_LAST)
        gemm::gemm_tile<gemm::EPI_FWD_LAST, false>(*ta, *tb, g, bx, p, smem, sh.g, tmem_base, g_slabs, g_tiles);
      else
        gemm::gemm_tile<gemm::EPI_DGRAD, false>(*ta, *tb, g, bx, p, smem, sh.g, tmem_base, g_slabs, g_tiles);
    }
    g_slabs += (uint32_t)g.nkb;
    g_tiles += 1;
    fence_proxy_async_all();               // this thread's results -> later TMA reads elsewhere
    tc_fence_before_sync();
    __syncthreads();
    if (sh.g.abort_flag) {
      stop = true;
      return;
    }
    if (threadIdx.x == 0)
      signal_done(counter(rp, kind == gemm::EPI_DGRAD ? CNT_D : CNT_F, l, p));
  };

  // ---- this block's share of a layer's weight-gradient + SGD tiles -------------------------------
  auto wgrad_unit = [&](int l, int k, int vb) {
    const RoundLayer& y = rp.ly[l];
    const bool shared_w = rp.first_shared && k == 1;
    wgrad::WgradArgs g{};
    g.w32_in_batched = shared_w ? 0 : 1;
    g.nkb = y.w_nkb; g.m_tiles = y.w_m_tiles; g.n_tiles = y.w_n_tiles;
    g.chunk = y.w_chunk; g.n_chunks = y.w_n_chunks;
    g.items = P * y.w_m_tiles * y.w_n_chunks;
    g.slots = rp.w_slots; g.a_bufs = rp.w_a_bufs; g.w16_on_b = rp.w_on_b;
    g.gamma = rp.gamma;
    g.keep_w32 = rp.keep_w32;
    g.status = rp.status;
    if (vb >= g.items) return;             // nothing of this layer falls to this block
    WgDeps dep{&rp, l, k};
    wgrad::wgrad_run<false>(rp.dz_t[l], l == 1 ? rp.x_in_t[k & 1] : rp.act_in_t[l], rp.w32[l],
                            shared_w ? rp.w32g[l] : rp.w32[l], rp.w16_st[l], rp.w32[l], g, vb, grid,
                            smem, sh.w, tmem_base, dep, w_tiles, w_items);
    wgrad::wgrad_run_totals(g, vb, grid, w_tiles, w_items);
    tc_fence_before_sync();
    __syncthreads();
    if (sh.w.abort_flag) stop = true;
  };

  // ---- a slice of the gather of step k -----------------------------------------------------------
  auto gather_unit = [&](int k, int t) {
    const int per_p = g_units(rp);
    const int p = t / per_p, u = t % per_p;
    const int sg = u / rp.g_col_splits, cs = u % rp.g_col_splits;
    if (threadIdx.x == 0) {
      if (!gather_deps(rp, p, k)) sh.stop = 1;
    }
    __syncthreads();
    if (sh.stop) {
      stop = true;
      return;
    }
    const int d = rp.ly[1].in;
    const int c_lo = cs * kGatherCols, c_hi = min(d, c_lo + kGatherCols);
    GatherStage& gs = *reinterpret_cast<GatherStage*>(smem);
    if (rp.x_bf16)
      gather_slice<__nv_bfloat16>(rp, gs, k, p, sg * 32, c_lo, c_hi, cs == 0);
    else
      gather_slice<float>(rp, gs, k, p, sg * 32, c_lo, c_hi, cs == 0);
    fence_proxy_async_all();
    __syncthreads();
    if (threadIdx.x == 0) signal_done(counter(rp, CNT_G, 0, p));
  };

  // first unit of a segment of n units that falls to this block; advances the rotation
  auto first_of = [&](int n) {
    const int v = ((cta - rot) % grid + grid) % grid;
    rot = (rot + n) % grid;
    return v;
  };

  const int n_gather = P * g_units(rp);
  if (!stop) {
    for (int t = first_of(n_gather); t < n_gather && !stop; t += grid) gather_unit(1, t);
  }
  for (int k = 1; k <= K && !stop; ++k) {
    // the same block runs the same units in every step: its instruction cache keeps their code
    rot = 0;
    for (int l = 1; l < L && !stop; ++l) {
      const int n = P * f_tiles(rp.ly[l]);
      for (int t = first_of(n); t < n && !stop; t += grid) gemm_unit(gemm::EPI_FWD_HIDDEN, l, k, t);
    }
    {
      const int n = P;                      // the last layer has one tile per learner
      const int rot_fl = rot;
      for (int t = first_of(n); t < n && !stop; t += grid) gemm_unit(gemm::EPI_FWD_LAST, L, k, t);
      if (k < K) {
        // The next step's gather runs beside the narrow tail of this step (last layer, the first
        // dgrad products).  Where those leave at least half of the blocks idle, the gather goes
        // to the idle ones only, so that it never delays a unit the step is waiting for.
        int n_crit = P + P * rp.ly[L].d_m_tiles + (L >= 3 ? P * rp.ly[L - 1].d_m_tiles : 0);
        if (n_crit <= grid / 2) {
          const int gw = grid - n_crit;
          const int gi = ((cta - rot_fl - n_crit) % grid + grid) % grid;
          if (gi < gw)
            for (int t = gi; t < n_gather && !stop; t += gw) gather_unit(k + 1, t);
        } else {
          for (int t = first_of(n_gather); t < n_gather && !stop; t += grid) gather_unit(k + 1, t);
        }
      }
    }
    for (int l = L; l >= 2 && !stop; --l) {
      const int n = P * rp.ly[l].d_m_tiles;
      for (int t = first_of(n); t < n && !stop; t += grid) gemm_unit(gemm::EPI_DGRAD, l, k, t);
      if (l < L && !stop) {
        const int items = P * wg_items(rp.ly[l + 1]);
        wgrad_unit(l + 1, k, first_of(items));
      }
    }
    for (int l = min(2, L); l >= 1 && !stop; --l) {
      const int items = P * wg_items(rp.ly[l]);
      wgrad_unit(l, k, first_of(items));
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 256);
}

}  // namespace

bool tc_round_supported(mavg_ctx* c) {
  const TcState* st = (const TcState*)c->mlp;
  const mavg_config& cfg = c->cfg;
  if (!st || !st->round_ok) return false;
  if (cfg.learner_momentum != 0.f) return false;
  return true;
}

// Decides once per handle whether the whole-round kernel covers the problem, and sizes it.
cudaError_t tc_round_prepare(mavg_ctx* c) {
  TcState* st = (TcState*)c->mlp;
  const mavg_config& cfg = c->cfg;
  st->round_ok = false;
  const int L = cfg.n_layers;
  if (L < 2 || L > kRoundMaxLayers) return cudaSuccess;
  int stages = gemm::kMaxStages;
  size_t smem = 0;
  for (int l = 1; l <= L; ++l) {
    const GemmPlan& f = st->fwd[l];
    if (f.splits != 1) return cudaSuccess;
    stages = std::min(stages, f.stages);
    if (l > 1) {
      if (st->dgrad[l].splits != 1) return cudaSuccess;
      stages = std::min(stages, st->dgrad[l].stages);
    }
    if (st->wgrad[l].slots != st->wgrad[1].slots || st->wgrad[l].a_bufs != st->wgrad[1].a_bufs)
      return cudaSuccess;
    smem = std::max(smem, st->wgrad[l].smem);
  }
  if (stages < 2) return cudaSuccess;
  for (int l = 1; l <= L; ++l) {
    smem = std::max(smem, (size_t)stages * (gemm::kATileBytes + st->fwd[l].BN * gemm::kBK * 2) + 1024);
    if (l > 1)
      smem = std::max(smem, (size_t)stages * (gemm::kATileBytes + st->dgrad[l].BN * gemm::kBK * 2) + 1024);
  }
  // the loss tail keeps logits, dZ and the row losses in the pipeline buffer
  smem = std::max(smem, ((size_t)2 * cfg.B * cfg.dims[L] + cfg.B) * sizeof(float) + 1024);
  smem = std::max(smem, sizeof(GatherStage) + 1024);
  int coop = 0, dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  if (e != cudaSuccess) return e;
  if (!coop) return cudaSuccess;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, k_mlp_round);
  if (e != cudaSuccess) return e;
  if (smem + fa.sharedSizeBytes > 227 * 1024) return cudaSuccess;
  e = cudaFuncSetAttribute(k_mlp_round, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_mlp_round, kRoundThreads, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaSuccess;
  st->round_stages = stages;
  st->round_smem = smem;
  st->round_grid = c->sm_count;
  st->round_ok = true;
  return cudaSuccess;
}

cudaError_t tc_round_launch(mavg_ctx* c, int64_t round) {
  TcState* st = (TcState*)c->mlp;
  const TcLayout& t = st->lay;
  const mavg_config& cfg = c->cfg;
  const int L = cfg.n_layers, P = cfg.P, B = cfg.B;
  char* ws = (char*)c->buf.workspace;
  auto bfp = [&](size_t off) { return (__nv_bfloat16*)(ws + off); };
  static_assert(sizeof(RoundParams) < 16 * 1024, "kernel parameter block too large");
  RoundParams* rp = new RoundParams();
  for (int l = 1; l <= L; ++l) {
    rp->w[l] = st->w[l]; rp->wg[l] = st->wg[l];
    rp->w_mn[l] = st->w_mn[l]; rp->wg_mn[l] = st->wg_mn[l];
    rp->act_in[l] = st->act_in[l]; rp->act_in_t[l] = st->act_in_t[l];
    rp->dz[l] = st->dz[l]; rp->dz_t[l] = st->dz_t[l];
    rp->w32[l] = st->w32[l]; rp->w32g[l] = st->w32g[l]; rp->w16_st[l] = st->w16_st[l];
    if (l == st->dbl_layer && st->w16_cur == 1) {   // the copy that holds this layer's weights now
      rp->w[l] = st->w_b; rp->w_mn[l] = st->w_mn_b; rp->w16_st[l] = st->w16_st_b;
    }
    RoundLayer& y = rp->ly[l];
    const MlpLayer& ml = c->layers[l - 1];
    y.in = ml.in; y.out = ml.out; y.w_off = ml.w_off; y.b_off = ml.b_off;
    const GemmPlan& f = st->fwd[l];
    y.f_BN = f.BN; y.f_m_tiles = f.m_tiles; y.f_n_tiles = f.n_tiles; y.f_nkb = f.nkb;
    if (l > 1) {
      const GemmPlan& d = st->dgrad[l];
      y.d_BN = d.BN; y.d_m_tiles = d.m_tiles; y.d_nkb = d.nkb;
    }
    const WgradPlan& w = st->wgrad[l];
    y.w_nkb = w.nkb; y.w_m_tiles = w.m_tiles; y.w_n_tiles = w.n_tiles; y.w_chunk = w.chunk;
    y.w_n_chunks = w.n_chunks;
    if (l < L) { y.act = bfp(t.act[l]); y.act_t = bfp(t.act_t[l]); }
    y.dz = bfp(t.dz[l]); y.dz_t = bfp(t.dz_t[l]);
  }
  for (int i = 0; i < 2; ++i) {
    rp->x_in[i] = st->x_in[i]; rp->x_in_t[i] = st->x_in_t[i];
    rp->xg[i] = bfp(t.xg[i]); rp->xt[i] = bfp(t.xt[i]);
  }
  rp->L = L; rp->P = P; rp->B = B; rp->K = cfg.K; rp->cpad = t.cpad;
  rp->first_shared = c->replicas_equal_global ? 1 : 0;
  rp->stages = st->round_stages;
  rp->w_slots = st->wgrad[1].slots; rp->w_a_bufs = st->wgrad[1].a_bufs;
  rp->w_on_b = st->wgrad[1].w16_on_b;
  rp->g_slot_groups = (B + 31) / 32;
  rp->g_col_splits = (cfg.dims[0] + kGatherCols - 1) / kGatherCols;
  rp->round = round; rp->seed = cfg.seed; rp->S = cfg.n_samples;
  rp->x = cfg.x; rp->x_bf16 = cfg.x_dtype == MAVG_X_BF16 ? 1 : 0; rp->y = cfg.y;
  // labels of odd steps live in the labels buffer, of even steps in the index buffer (the index
  // stream itself is not kept by this kernel)
  rp->labels[1] = (int32_t*)ws_ptr(c, c->ws.labels);
  rp->labels[0] = (int32_t*)ws_ptr(c, c->ws.idx);
  rp->losses = (float*)ws_ptr(c, c->ws.losses);
  rp->replicas = c->buf.replicas; rp->global_w = c->buf.global_w;
  rp->rep_stride = c->buf.replica_stride;
  rp->gamma = cfg.local_lr;
  rp->keep_w32 = c->l2_keep ? 1 : 0;
  rp->counters = (int*)(ws + t.round_ctr);
  rp->status = (int*)ws_ptr(c, c->ws.status);
  cudaError_t e = cudaMemsetAsync(rp->counters, 0, t.round_ctr_bytes, c->stream);
  if (e == cudaSuccess) {
    void* args[] = {(void*)rp};
    prof_begin(c, MAVG_K_FWD);
    e = cudaLaunchCooperativeKernel((const void*)k_mlp_round, dim3((unsigned)st->round_grid),
                                    dim3(kRoundThreads), args, st->round_smem, c->stream);
    prof_end(c);
  }
  delete rp;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace mavg
