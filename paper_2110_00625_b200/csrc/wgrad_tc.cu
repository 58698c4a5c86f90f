// Weight gradient fused with the SGD step of Algorithm 1, as a persistent streaming kernel:
//   W[o, i] <- W[o, i] - gamma * sum_b dZ[b, o] A[b, i]          (fp32 masters, per learner)
// and the refreshed bf16 copy of W that the forward and dgrad products read.
//
// The contraction is only as long as the batch, so the kernel is a read-modify-write stream over
// the masters (10 bytes per weight) and is built around bulk copies, not around the MMA:
//   producer warp   TMA-loads, per 128 x 32 weight tile, the fp32 master tile and the 32 x B tile
//                   of A^T into a ring of shared-memory slots; the 128 x B tile of dZ^T is loaded
//                   once per work item (a run of column tiles of one learner and row tile);
//   MMA warp        one thread issues tcgen05.mma (M=128, N=32, K=B) into one of two TMEM buffers;
//   2 x 4 epilogue warps (one group per TMEM buffer, i.e. per tile parity) read the accumulator
//                   (tcgen05.ld, one weight row per lane), update the master tile in place in
//                   shared memory and write the bf16 tile beside it;
//   store warp      one thread sends the two finished tiles back with TMA stores and frees the
//                   slot once they have left shared memory.
// With learner-level momentum (MOM) the tile of u^j travels with the master tile: loaded into the
// same slot (unless the momentum is reset at this step), updated in place (u <- beta u - gamma dW;
// W <- W + u) and stored back, 18 bytes per weight instead of 10.
// Edge tiles need no predicates: TMA zero-fills loads and clips stores at the tensor bounds.
//
// The 512-thread instantiation (FWD) lets the NEXT local step's forward product of the same layer
// ride along: the epilogue has just put the updated bf16 tile W16[128, 32] into the slot, and the
// producer has loaded the matching [B, 32] tile of the next step's input Xn beside it, so
//   forward warp    one thread issues W16_tile . Xn_tile^T (M=128, N=B, K=32) into a third TMEM
//                   accumulator that collects a whole run of column tiles; the slot is released
//                   only after these MMAs have read it;
//   4 more warps    read that accumulator once per run.  A run that covers its whole row adds the
//                   bias, applies ReLU and writes the next step's activations (bf16, both
//                   orientations) at once; the runs of a row that is cut leave fp32 partial sums
//                   and bump the row's arrival counter, and the one that arrives last adds the
//                   partial sums in ascending run order and finishes the row.
// Per weight and step this removes the forward product's read of the bf16 copy and, for a layer
// without a dgrad product (layer 1), the copy itself.
#include <cuda.h>

#include <algorithm>

#include "mlp.cuh"
#include "tc_ptx.cuh"
#include "wgrad_tc.cuh"
#include "wgrad_unit.cuh"

namespace mavg {
namespace {

using namespace tc;
using namespace wgrad;

template <bool MOM, bool FWD>
__global__ void __launch_bounds__(FWD ? kThreadsFwd : kThreads)
k_wgrad_sgd_stream(const __grid_constant__ CUtensorMap tm_dzt,   // bf16 [P, out, B]  load
                   const __grid_constant__ CUtensorMap tm_at,    // bf16 [P, in, B]   load
                   const __grid_constant__ CUtensorMap tm_w32,   // fp32 [P, out, in] store
                   const __grid_constant__ CUtensorMap tm_w32_in,  // fp32 masters to load: the same
                                                                   // array, or w~ [1, out, in] at
                                                                   // the first step of a round
                   const __grid_constant__ CUtensorMap tm_w16,   // bf16 [P, out, in] store
                   const __grid_constant__ CUtensorMap tm_u,     // fp32 [P, out, in] u^j, load + store (MOM)
                   const __grid_constant__ CUtensorMap tm_xn,    // bf16 [P, B, in] next step's input (fwd_next)
                   const WgradArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) WgradShared sh;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5;

  grid_launch_dependents();
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tm_dzt);
    tma_prefetch_desc(&tm_at);
    tma_prefetch_desc(&tm_w32);
    tma_prefetch_desc(&tm_w32_in);
    tma_prefetch_desc(&tm_w16);
    if (MOM) tma_prefetch_desc(&tm_u);
    if (FWD && g.fwd_next) tma_prefetch_desc(&tm_xn);
    wgrad_init_barriers(sh, g.slots);
    sh.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  // two accumulators of 32 columns; with fwd_next a third of B columns behind them
  const uint32_t tmem_cols = !(FWD && g.fwd_next) ? 64u : (g.batch <= 64 ? 128u : 256u);
  if (warp == 1) {
    tmem_alloc(&sh.tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh.tmem_slot;
  grid_dependency_wait();
  wgrad_run<MOM, FWD>(tm_dzt, tm_at, tm_w32, tm_w32_in, tm_w16, tm_u, tm_xn, g, (int)blockIdx.x,
                 (int)gridDim.x, smem, sh, tmem_base);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
}

// The same for several layers in one launch: every block makes one run per layer, in the order
// given, with the ring and its barriers carried from run to run (all layers share the batch, so
// their rings have the same geometry).  For workloads whose single layers are too small to pay
// for a persistent launch each.
struct WgradMultiParams {
  CUtensorMap dzt[MAVG_MAX_LAYERS], at[MAVG_MAX_LAYERS], w32[MAVG_MAX_LAYERS],
      w32_in[MAVG_MAX_LAYERS], w16[MAVG_MAX_LAYERS], u[MAVG_MAX_LAYERS];
  WgradArgs g[MAVG_MAX_LAYERS];
  int rot[MAVG_MAX_LAYERS];    // block b takes the items (b + rot) % grid, + grid, ... of a layer
  int n;
};

template <bool MOM>
__global__ void __launch_bounds__(kThreads)
k_wgrad_sgd_multi(const __grid_constant__ WgradMultiParams mp) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) WgradShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5;
  grid_launch_dependents();
  if (threadIdx.x == 0) {
    wgrad_init_barriers(sh, mp.g[0].slots);
    sh.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_slot, 64);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh.tmem_slot;
  grid_dependency_wait();
  uint32_t tiles = 0, items = 0;
  const int grid = (int)gridDim.x;
  for (int s = 0; s < mp.n; ++s) {
    const int vb = ((int)blockIdx.x + mp.rot[s]) % grid;
    wgrad_run<MOM, false>(mp.dzt[s], mp.at[s], mp.w32[s], mp.w32_in[s], mp.w16[s], mp.u[s], mp.w16[s],
                   mp.g[s], vb, grid, smem, sh, tmem_base, tiles, items);
    wgrad_run_totals(mp.g[s], vb, grid, tiles, items);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 64);
}

}  // namespace

// longest run of column tiles of one work item
#ifndef MAVG_WGRAD_CHUNK_CAP
#define MAVG_WGRAD_CHUNK_CAP 16
#endif
constexpr long kWgradChunkCap = MAVG_WGRAD_CHUNK_CAP;
// deepest ring the plan may choose (at most kMaxSlots)
#ifndef MAVG_WGRAD_SLOT_CAP
#define MAVG_WGRAD_SLOT_CAP 6
#endif
// the same two for a launch that streams its masters through HBM
#ifndef MAVG_WGRAD_STREAM_CHUNK
#define MAVG_WGRAD_STREAM_CHUNK 8
#endif
#ifndef MAVG_WGRAD_STREAM_SLOTS
#define MAVG_WGRAD_STREAM_SLOTS 4
#endif
constexpr long kWgradStreamChunk = MAVG_WGRAD_STREAM_CHUNK;
#ifndef MAVG_WGRAD_FWD_SLOTS
#define MAVG_WGRAD_FWD_SLOTS 6
#endif
constexpr int kWgradFwdSlots = MAVG_WGRAD_FWD_SLOTS;
constexpr int kWgradStreamSlots = MAVG_WGRAD_STREAM_SLOTS;
constexpr int kWgradSlotCap = MAVG_WGRAD_SLOT_CAP < wgrad::kMaxSlots ? MAVG_WGRAD_SLOT_CAP : wgrad::kMaxSlots;

WgradPlan plan_wgrad_stream(int out, int in, int B, int P, int sm_count, bool momentum,
                            bool streaming, bool fwd_next) {
  WgradPlan w{};
  w.nkb = (B + kBK - 1) / kBK;
  w.m_tiles = (out + kBM - 1) / kBM;
  w.n_tiles = (in + kBN - 1) / kBN;
  const long total = (long)P * w.m_tiles * w.n_tiles;
  long chunk = total / (5L * sm_count);
  if (chunk < 1) chunk = 1;
  if (chunk > kWgradChunkCap) chunk = kWgradChunkCap;
  if (streaming && chunk > kWgradStreamChunk) chunk = kWgradStreamChunk;
  // With a riding forward product every run ends with per-run work -- reading the forward
  // accumulator, the partial sum and its share of the sums over all runs of a row, during which
  // the next run's forward products wait -- worth about eight tile periods (measured with 8
  // learners: runs of 8 tiles took 150 us per launch where runs of 32 to 48 take 75 us).  So: as
  // many whole waves of whole rows as pay (one item per (learner, row tile), no partial sums at
  // all), then the remaining rows cut evenly into runs of at least 16 tiles; taken is the
  // combination whose busiest block finishes first.
  long whole_rows = 0;
  if (fwd_next) {
    const long rows = (long)P * w.m_tiles, per_run = 8;
    long best_cost = -1;
    for (long waves = 0; waves * sm_count <= rows; ++waves) {
      const long rest = rows - waves * sm_count;
      const long head = waves * (w.n_tiles + per_run);
      if (rest == 0) {
        if (best_cost < 0 || head < best_cost) { best_cost = head; whole_rows = rows; chunk = w.n_tiles; }
        break;
      }
      for (int nc = 1; nc <= w.n_tiles; ++nc) {
        const long run = (w.n_tiles + nc - 1) / nc;
        if (run < 16 && nc > 1) break;
        const long items = rest * ((w.n_tiles + run - 1) / run);
        const long cost = head + ((items + sm_count - 1) / sm_count) * (run + per_run);
        if (best_cost < 0 || cost < best_cost) {
          best_cost = cost;
          whole_rows = waves * sm_count;
          chunk = run;
        }
      }
    }
  }
  if (chunk > w.n_tiles) chunk = w.n_tiles;
  w.chunk = (int)chunk;
  w.n_chunks = (w.n_tiles + w.chunk - 1) / w.chunk;
  w.whole_rows = (int)whole_rows;
  w.items = w.whole_rows + (P * w.m_tiles - w.whole_rows) * w.n_chunks;
  const int a_bytes = w.nkb * kBM * kBK * 2;
  const int b_bytes = w.nkb * kBN * kBK * 2;
  w.w16_on_b = b_bytes >= kW16Bytes ? 1 : 0;   // the bf16 output tile reuses the A^T slabs' space
  w.xn_bytes = fwd_next ? B * kBN * 2 : 0;
  const int slot_bytes = kW32Bytes + (momentum ? kW32Bytes : 0) + (w.w16_on_b ? 0 : kW16Bytes) +
                         b_bytes + w.xn_bytes;
  const int budget = 220 * 1024;
  w.a_bufs = 2;
  w.slots = (budget - 2 * a_bytes) / slot_bytes;
  if (w.slots < 2) {
    w.a_bufs = 1;
    w.slots = (budget - a_bytes) / slot_bytes;
  }
  if (w.slots > kWgradSlotCap) w.slots = kWgradSlotCap;
  const int stream_slots = fwd_next ? kWgradFwdSlots : kWgradStreamSlots;
  if (streaming && w.slots > stream_slots) w.slots = stream_slots;
  w.smem = (size_t)w.a_bufs * a_bytes + (size_t)w.slots * slot_bytes + 1024;
  w.grid = w.items < sm_count ? w.items : sm_count;
  return w;
}

cudaError_t wgrad_stream_prepare() {
  const void* kernels[] = {(const void*)k_wgrad_sgd_stream<false, false>,
                           (const void*)k_wgrad_sgd_stream<true, false>,
                           (const void*)k_wgrad_sgd_stream<false, true>,
                           (const void*)k_wgrad_sgd_stream<true, true>,
                           (const void*)k_wgrad_sgd_multi<false>,
                           (const void*)k_wgrad_sgd_multi<true>};
  for (const void* k : kernels) {
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

namespace {
WgradArgs make_args(mavg_ctx* c, const WgradPlan& w, bool shared, const MomArgs& mom) {
  WgradArgs g{};
  g.w32_in_batched = shared ? 0 : 1;
  g.nkb = w.nkb;
  g.m_tiles = w.m_tiles;
  g.n_tiles = w.n_tiles;
  g.chunk = w.chunk;
  g.n_chunks = w.n_chunks;
  g.items = w.items;
  g.whole_rows = w.whole_rows;
  g.slots = w.slots;
  g.a_bufs = w.a_bufs;
  g.w16_on_b = w.w16_on_b;
  g.keep_w32 = c->l2_keep ? 1 : 0;
  g.gamma = c->cfg.local_lr;
  g.beta = mom.beta;
  g.read_u = mom.read_u;
  g.fwd_next = 0;
  g.store_w16 = 1;
  g.xn_bytes = w.xn_bytes;
  g.batch = c->cfg.B;
  g.zpart = nullptr;
  g.status = (int*)ws_ptr(c, c->ws.status);
  return g;
}
}  // namespace

cudaError_t launch_wgrad_multi(mavg_ctx* c, int n, const WgradLayerRef* layers, const MomArgs& mom,
                               int max_grid) {
  WgradMultiParams* mp = new WgradMultiParams();
  mp->n = n;
  int grid = 1, rot = 0;
  size_t smem = 0;
  for (int s = 0; s < n; ++s) grid = layers[s].plan->grid > grid ? layers[s].plan->grid : grid;
  if (max_grid > 0 && grid > max_grid) grid = max_grid;
  const bool with_u = mom.u != nullptr;
  for (int s = 0; s < n; ++s) {
    const WgradLayerRef& r = layers[s];
    mp->dzt[s] = *r.dzt; mp->at[s] = *r.at; mp->w32[s] = *r.w32;
    mp->w32_in[s] = r.w32_shared ? *r.w32_shared : *r.w32;
    mp->w16[s] = *r.w16;
    mp->u[s] = (with_u && r.u32) ? *r.u32 : *r.w32;
    mp->g[s] = make_args(c, *r.plan, r.w32_shared != nullptr, mom);
    mp->rot[s] = (grid - rot % grid) % grid;   // this layer's item 0 goes to block `rot`
    rot = (rot + r.plan->items) % grid;
    smem = r.plan->smem > smem ? r.plan->smem : smem;
  }
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)grid);
  lc.blockDim = dim3(kThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at_[1];
  at_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at_[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at_;
  lc.numAttrs = 1;
  prof_begin(c, MAVG_K_WGRAD_SGD);
  cudaError_t e = with_u ? cudaLaunchKernelEx(&lc, k_wgrad_sgd_multi<true>, *mp)
                         : cudaLaunchKernelEx(&lc, k_wgrad_sgd_multi<false>, *mp);
  prof_end(c);
  delete mp;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_wgrad_stream(mavg_ctx* c, const WgradPlan& w, const CUtensorMap& dzt,
                                const CUtensorMap& at, const CUtensorMap& w32,
                                const CUtensorMap& w16, const CUtensorMap* w32_shared,
                                const CUtensorMap* u32, const MomArgs& mom,
                                const WgradFwdNext* fn) {
  WgradArgs g = make_args(c, w, w32_shared != nullptr, mom);
  if (fn) {
    // the plan must have been made with fwd_next (room for the input tile in every slot)
    if (w.xn_bytes == 0 || !fn->xn) return cudaErrorInvalidValue;
    g.fwd_next = 1;
    g.store_w16 = fn->store_w16 ? 1 : 0;
    g.zpart = fn->zpart;
    g.zcount = fn->zcount;
    g.bias_rep = c->buf.replicas;
    g.rep_stride = c->buf.replica_stride;
    g.bias_off = fn->bias_off;
    g.out_rows = fn->out_rows;
    g.out_bm = fn->out_bm;
    g.out_mb = fn->out_mb;
  } else {
    g.xn_bytes = w.xn_bytes;   // the slot keeps its shape; the tile is simply not loaded
  }
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)w.grid);
  lc.blockDim = dim3(fn ? kThreadsFwd : kThreads);
  lc.dynamicSmemBytes = w.smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at_[1];
  at_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at_[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at_;
  lc.numAttrs = 1;
  const bool with_u = mom.u && u32;
  const CUtensorMap& w32_in = w32_shared ? *w32_shared : w32;
  const CUtensorMap& um = with_u ? *u32 : w32;
  prof_begin(c, MAVG_K_WGRAD_SGD);
  cudaError_t e;
  if (fn)
    e = with_u ? cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<true, true>, dzt, at, w32, w32_in, w16, um, *fn->xn, g)
               : cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<false, true>, dzt, at, w32, w32_in, w16, um, *fn->xn, g);
  else
    e = with_u ? cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<true, false>, dzt, at, w32, w32_in, w16, um, w16, g)
               : cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<false, false>, dzt, at, w32, w32_in, w16, um, w16, g);
  prof_end(c);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace mavg
