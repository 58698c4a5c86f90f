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

#include "gemm_unit.cuh"
#include "mlp.cuh"
#include "tc_ptx.cuh"
#include "tc_state.cuh"
#include "wgrad_tc.cuh"

namespace mavg {
namespace {

using namespace tc;

constexpr int kThreads = 320;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
using namespace gemm;

// MINB = 2 caps the registers so that two blocks fit an SM (used when a launch has more blocks
// than SMs; costs a few spills in the tail), MINB = 1 leaves the compiler free.
template <int EPI, int MINB>
__global__ void __launch_bounds__(kThreads, MINB)
k_tc_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
          const TcArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) GemmShared sh;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5;

  grid_launch_dependents();   // the next kernel may begin its own set-up early
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    gemm_init_barriers(sh, g.stages);
    sh.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_slot, g.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh.tmem_slot;
  // Everything above touched only this block's own shared and tensor memory.  When the launch
  // allowed it, that much ran while the previous kernel of the stream was still finishing; from
  // here on its results are read, so wait for it to complete (returns at once otherwise).
  grid_dependency_wait();
  // the split path is compiled out of the register-capped build, which is never used with a split
  gemm_tile<EPI, MINB == 1>(tmA, tmB, g, (int)blockIdx.x, (int)blockIdx.y, smem, sh, tmem_base);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, g.tmem_cols);
}

// Hidden-layer forward tile with its contraction split over the blocks of a cluster (see
// gemm_tile, CLUSTER): grid.x = row tiles x splits, cluster = the `splits` blocks of a row tile.
__global__ void __launch_bounds__(kThreads, 1)
k_tc_gemm_ks(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const TcArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) GemmShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5;
  grid_launch_dependents();
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    gemm_init_barriers(sh, g.stages);
    // every lane of the four sending warps of each other block arrives once
    mbar_init(&sh.recv_bar, (uint32_t)(g.splits - 1) * 128u);
    sh.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_slot, g.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  cluster_sync_all();           // every block's barriers exist before anyone arrives on them
  const uint32_t tmem_base = sh.tmem_slot;
  grid_dependency_wait();
  gemm_tile<EPI_FWD_HIDDEN, false, true>(tmA, tmB, g, (int)blockIdx.x, (int)blockIdx.y, smem, sh,
                                         tmem_base);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();           // nobody leaves while a peer may still write into its shared memory
  if (warp == 1) tmem_dealloc(tmem_base, g.tmem_cols);
}

// bf16 copy of the global model w~ (shared by all learners at the first step of a round, when
// every replica equals w~).  One launch for all layers: block row y takes layer y, grid-stride
// over that layer's weights.
struct ShadowArgs {
  int64_t w_off[MAVG_MAX_LAYERS], total[MAVG_MAX_LAYERS], sh_off[MAVG_MAX_LAYERS];
};
__global__ void __launch_bounds__(256)
k_shadow_from_global(const float* __restrict__ w, __nv_bfloat16* __restrict__ w16,
                     const ShadowArgs a) {
  const int l = blockIdx.y;
  const float* src = w + a.w_off[l];
  __nv_bfloat16* dst = w16 + a.sh_off[l];
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < a.total[l];
       t += (int64_t)gridDim.x * blockDim.x)
    dst[t] = __float2bfloat16_rn(src[t]);
}

// ---------------------------------------------------------------------------------- host side
size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

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
      t.act_b[l] = take(rows * d * 2);
      t.act_t_b[l] = take(rows * d * 2);
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
  t.tail_part = take(tail_fused_supported(cfg) ? tail_fused_part_bytes(cfg) : 16);
  {
    // partial sums of a forward product that rides along with a weight-gradient launch: one
    // 128 x B fp32 tile per (learner, row tile, run of column tiles) of that launch's plan; the
    // layers use the space one after the other
    t.zpart_bytes = 16;
    t.zcount_bytes = 16;
    if (B <= 128)
      for (int l = 1; l < L; ++l) {
        const WgradPlan w = plan_wgrad_stream(cfg->dims[l], cfg->dims[l - 1], B, P, sm_count, false, true, true);
        t.zpart_bytes = std::max(t.zpart_bytes, (size_t)P * w.m_tiles * w.n_chunks * B * kBM * sizeof(float));
        t.zcount_bytes = std::max(t.zcount_bytes, (size_t)P * w.m_tiles * sizeof(int));
      }
    t.zcount = take(t.zcount_bytes);
    t.zpart = take(t.zpart_bytes);
  }
  t.w16b_stride = L >= 3 ? (int64_t)up((size_t)cfg->dims[L - 2] * cfg->dims[L - 1], 64) : 0;
  t.w16b = take(L >= 3 ? (size_t)P * t.w16b_stride * 2 : 16);
  t.end = off;
  return t;
}

// SM count the plans (and with them the size of the partial buffer) are made for, so that the
// workspace size does not depend on the device that later runs the problem.
constexpr int kPlanSmCount = 148;

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

// Plan of the cluster-split forward product of a hidden layer, or splits = 1 if it does not apply:
// the default plan would cut the batch into B / 32 column tiles (so every block would stream the
// whole weight tile for a quarter or half of the batch), and the contraction is long enough.
GemmPlan plan_cluster_split(const GemmPlan& f, int M, int B, int K) {
  GemmPlan ks{};
  ks.splits = 1;
  const int S = B / 32;
  if ((B != 64 && B != 128) || f.splits != 1 || f.n_tiles != S || f.BN != 32) return ks;
  const int nkb = (K + kBK - 1) / kBK;
  const int per = (nkb + S - 1) / S;
  if (nkb < 4 * S || per * (S - 1) >= nkb) return ks;
  ks.BN = B;
  ks.m_tiles = (M + kBM - 1) / kBM;
  ks.n_tiles = 1;
  ks.nkb = nkb;
  ks.splits = S;
  ks.kb_per_split = per;
  const int stage_bytes = kATileBytes + B * kBK * 2;
  ks.stages = (216 * 1024 - S * kBM * 32 * 4) / stage_bytes;
  if (ks.stages > kMaxStages) ks.stages = kMaxStages;
  if (ks.stages > per) ks.stages = per;
  if (ks.stages < 2) { ks.splits = 1; return ks; }
  ks.tmem_cols = 32;
  while ((int)ks.tmem_cols < B) ks.tmem_cols <<= 1;
  return ks;
}

cudaError_t launch_gemm_ks(mavg_ctx* c, const CUtensorMap& a, const CUtensorMap& b,
                           const GemmPlan& pl, TcArgs g) {
  g.BN = pl.BN;
  g.m_tiles = pl.m_tiles;
  g.n_tiles = 1;
  g.splits = pl.splits;
  g.kb_per_split = pl.kb_per_split;
  g.nkb = pl.nkb;
  g.stages = pl.stages;
  g.tmem_cols = pl.tmem_cols;
  g.P = c->cfg.P;
  g.rep_stride = c->buf.replica_stride;
  g.gamma = c->cfg.local_lr;
  g.status = (int*)ws_ptr(c, c->ws.status);
  const size_t smem = (size_t)pl.stages * (kATileBytes + pl.BN * kBK * 2) +
                      (size_t)pl.splits * kBM * 32 * 4 + 1024;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)(pl.m_tiles * pl.splits), (unsigned)c->cfg.P);
  lc.blockDim = dim3(kThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = (unsigned)pl.splits;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  lc.attrs = at;
  lc.numAttrs = 2;
  prof_begin(c, MAVG_K_FWD);
  cudaError_t e = cudaLaunchKernelEx(&lc, k_tc_gemm_ks, a, b, g);
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
    st->fwd_ks[l] = GemmPlan{};
    st->fwd_ks[l].splits = 1;
    if (l < L) st->fwd_ks[l] = plan_cluster_split(st->fwd[l], out, B, in);
    st->wgrad_mom = c->buf.learner_u != nullptr;
    st->wgrad[l] = plan_wgrad_stream(out, in, B, P, c->sm_count, st->wgrad_mom, !masters_fit_l2(c));
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
    if (L >= 3 && l == L - 1) {      // second copy of this layer's bf16 weights
      st->dbl_layer = l;
      __nv_bfloat16* wb = (__nv_bfloat16*)bf(t.w16b);
      ok = ok && encode_map(st, &st->w_b, wb, in, out, P, in, t.w16b_stride, kBM, &why);
      ok = ok && encode_map(st, &st->w_mn_b, wb, in, out, P, in, t.w16b_stride, 64, &why);
      ok = ok && encode_any(st, &st->w16_st_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, wb, in, out, P,
                            in, t.w16b_stride, kWgradTileCols, kWgradTileRows,
                            CU_TENSOR_MAP_SWIZZLE_64B, &why);
    }
    ok = ok && encode_map(st, &st->wg_mn[l], w16g, in, out, 1, in, t.n16, 64, &why);
    if (l == 1) {
      for (int i = 0; i < 2 && ok; ++i) {
        ok = ok && encode_map(st, &st->x_in[i], bf(t.xg[i]), in, B, P, in, (int64_t)B * in,
                              st->fwd[l].BN, &why);
        ok = ok && encode_map(st, &st->x_in_t[i], bf(t.xt[i]), B, in, P, B, (int64_t)B * in,
                              kWgradTileCols, &why);
        if (st->fwd_ks[l].splits > 1)
          ok = ok && encode_map(st, &st->x_in_ks[i], bf(t.xg[i]), in, B, P, in, (int64_t)B * in,
                                B, &why);
      }
    } else {
      ok = ok && encode_map(st, &st->act_in[l], bf(t.act[l - 1]), in, B, P, in, (int64_t)B * in,
                            st->fwd[l].BN, &why);
      ok = ok && encode_map(st, &st->act_in_t[l], bf(t.act_t[l - 1]), B, in, P, B,
                            (int64_t)B * in, kWgradTileCols, &why);
      if (st->fwd_ks[l].splits > 1)
        ok = ok && encode_map(st, &st->act_in_ks[l], bf(t.act[l - 1]), in, B, P, in,
                              (int64_t)B * in, B, &why);
      // the same three views of the second set of activation buffers
      ok = ok && encode_map(st, &st->act_in_b[l], bf(t.act_b[l - 1]), in, B, P, in, (int64_t)B * in,
                            st->fwd[l].BN, &why);
      ok = ok && encode_map(st, &st->act_in_t_b[l], bf(t.act_t_b[l - 1]), B, in, P, B,
                            (int64_t)B * in, kWgradTileCols, &why);
      if (st->fwd_ks[l].splits > 1)
        ok = ok && encode_map(st, &st->act_in_ks_b[l], bf(t.act_b[l - 1]), in, B, P, in,
                              (int64_t)B * in, B, &why);
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
                           (const void*)k_tc_gemm<EPI_DGRAD, 1>,      (const void*)k_tc_gemm<EPI_DGRAD, 2>,
                           (const void*)k_tc_gemm_ks};
  for (const void* k : kernels)
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  if (e == cudaSuccess) e = wgrad_stream_prepare();
  // The fused CUDA-core last layer pays where the tensor-core products of that layer would leave
  // most of the GPU idle (few learners, narrow layer below); with many tiles the tensor-core
  // kernels are the faster ones.
  // Small problems (a few dozen weight tiles per SM in the largest layer): one persistent launch
  // takes the weight gradients of all layers, instead of one launch per layer on a side stream.
  {
    const WgradPlan& w1 = st->wgrad[1];
    st->wgrad_merged = L >= 2 && (long)P * w1.m_tiles * w1.n_tiles <= 64L * c->sm_count;
    for (int l = 2; l <= L; ++l)
      if (st->wgrad[l].slots != w1.slots || st->wgrad[l].a_bufs != w1.a_bufs) st->wgrad_merged = false;
  }
  // Where the weight gradients are launches of their own, the launch of layer l can take the
  // next step's forward product of layer l along (layers 1..fuse_upto, a prefix of the hidden
  // layers): its plan gets room for the next step's input tile and long runs, and the input
  // buffers get a view with 32-column boxes.
  st->fuse_upto = 0;
  if (!st->wgrad_merged && L >= 2 && B <= 128 && ok) {
    for (int l = 1; l < L; ++l) {
      const int in = cfg.dims[l - 1], out = cfg.dims[l];
      const WgradPlan w = plan_wgrad_stream(out, in, B, P, c->sm_count, st->wgrad_mom,
                                            !masters_fit_l2(c), true);
      const size_t need = (size_t)P * w.m_tiles * w.n_chunks * B * kBM * sizeof(float);
      if (w.slots < 2 || need > t.zpart_bytes || (size_t)P * w.m_tiles * sizeof(int) > t.zcount_bytes)
        break;
      bool enc = true;
      for (int i = 0; i < 2 && enc; ++i) {
        const size_t src = l == 1 ? t.xg[i] : (i == 0 ? t.act[l - 1] : t.act_b[l - 1]);
        enc = encode_any(st, &st->a_next[l][i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bf(src), in, B,
                         P, in, (int64_t)B * in, kWgradTileCols, B, CU_TENSOR_MAP_SWIZZLE_64B, &why);
      }
      if (!enc) break;
      st->wgrad_f[l] = w;
      st->fuse_upto = l;
    }
  }
  // First step of a round: the hidden layers' forward products as one dense product each, where
  // that gives enough tiles (the input buffers seen as one [P*B, in] array).
  for (int l = 1; l <= L; ++l) st->dense[l] = DensePlan{};
  for (int l = 1; l < L && ok; ++l) {
    const int in = cfg.dims[l - 1];
    DensePlan pl = plan_fwd_dense(cfg.dims[l], in, B, P, c->sm_count);
    if (!pl.ok) continue;
    bool enc = true;
    for (int i = 0; i < 2 && enc; ++i) {
      const size_t src = l == 1 ? t.xg[i] : (i == 0 ? t.act[l - 1] : t.act_b[l - 1]);
      enc = encode_map(st, &st->in2d[l][i], bf(src), in, P * B, 1, in, (int64_t)P * B * in,
                       kDenseCols, &why);
    }
    if (enc) st->dense[l] = pl;
  }
  if (e == cudaSuccess) e = fwd_dense_prepare();
  // the meta-update writes the bf16 copy of w~ itself where its vector kernel takes the whole model
  c->shadow.dst = (__nv_bfloat16*)(ws + t.w16g);
  c->shadow.L = L;
  for (int l = 1; l <= L; ++l) {
    c->shadow.w_off[l - 1] = c->layers[l - 1].w_off;
    c->shadow.total[l - 1] = (int64_t)c->layers[l - 1].in * c->layers[l - 1].out;
    c->shadow.sh_off[l - 1] = t.sh_off[l - 1];
  }
  st->tail_ok = tail_fused_supported(&cfg) &&
                P * ((cfg.dims[L - 1] + kBM - 1) / kBM) <= c->sm_count / 2;
  if (e == cudaSuccess && st->tail_ok) e = tail_fused_prepare();
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&st->s_wgrad, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&st->s_gather, cudaStreamNonBlocking);
  cudaEvent_t* evs[] = {&st->ev_fork, &st->ev_wgrad_done, &st->ev_gather_done, &st->ev_x_free[0],
                        &st->ev_x_free[1]};
  for (cudaEvent_t* ev : evs)
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ws + t.counters, 0, t.counters_bytes, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + t.zcount, 0, t.zcount_bytes, c->stream);

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

int tc_get_w16_cur(mavg_ctx* c) { return c->mlp ? ((TcState*)c->mlp)->w16_cur : 0; }
void tc_set_w16_cur(mavg_ctx* c, int cur) {
  if (c->mlp) ((TcState*)c->mlp)->w16_cur = cur;
}

// After an abandoned wait the arrival counters of split tiles and of riding forward products may
// have been left mid-count: zero them (stream-ordered), so that the handle's next launches count
// from a clean state.
void tc_reset_counters(mavg_ctx* c) {
  const TcState* st = (const TcState*)c->mlp;
  if (!st) return;
  char* ws = (char*)c->buf.workspace;
  cudaMemsetAsync(ws + st->lay.counters, 0, st->lay.counters_bytes, c->stream);
  cudaMemsetAsync(ws + st->lay.zcount, 0, st->lay.zcount_bytes, c->stream);
}

void tc_step_plan(mavg_ctx* c, int32_t* out) {
  const TcState* st = (const TcState*)c->mlp;
  if (!st) return;
  out[MAVG_PLAN_TENSOR_PATH] = 1;
  out[MAVG_PLAN_WGRAD_MERGED] = st->wgrad_merged ? 1 : 0;
  out[MAVG_PLAN_FWD_WITH_WGRAD] = st->fuse_upto;
  for (int l = 1; l <= st->fuse_upto; ++l) {
    out[MAVG_PLAN_FWD_RUN_TILES + l - 1] = st->wgrad_f[l].chunk;
    out[MAVG_PLAN_FWD_WHOLE_ROWS + l - 1] = st->wgrad_f[l].whole_rows;
  }
  for (int l = 1; l <= MAVG_MAX_LAYERS; ++l)
    if (st->dense[l].ok) out[MAVG_PLAN_DENSE_FIRST_STEP] |= 1 << (l - 1);
}

cudaError_t tc_refresh_shared_operands(mavg_ctx* c) {
  TcState* st = (TcState*)c->mlp;
  const TcLayout& t = st->lay;
  char* ws = (char*)c->buf.workspace;
  ShadowArgs a{};
  int64_t most = 0;
  for (int l = 1; l <= c->cfg.n_layers; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    a.w_off[l - 1] = ly.w_off;
    a.total[l - 1] = (int64_t)ly.in * ly.out;
    a.sh_off[l - 1] = t.sh_off[l - 1];
    most = std::max(most, a.total[l - 1]);
  }
  const int gx = (int)std::min<int64_t>((most + 255) / 256, (int64_t)c->sm_count * 4);
  prof_begin(c, MAVG_K_AUX);
  k_shadow_from_global<<<dim3((unsigned)gx, (unsigned)c->cfg.n_layers), 256, 0, c->stream>>>(
      c->buf.global_w, (__nv_bfloat16*)(ws + t.w16g), a);
  prof_end(c);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
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
  const bool fused_tail = st->tail_ok && c->schedule == 0;
  bool tail_on_side = false;
  const bool merged = st->wgrad_merged && c->schedule == 0;
  // Forward products of the NEXT step ride along with this step's weight-gradient launches of
  // layers 1..ride (default schedule, those launches standing alone, a next step in this call);
  // the step after finds the activations of its first fwd_done layers in place.
  const int ride = (c->schedule == 0 && !merged && step < K) ? st->fuse_upto : 0;
  const int done = step == 1 ? 0 : st->fwd_done;
  st->fwd_done = 0;
  // activation buffers of this step and of the next
  const int ab = st->fuse_upto >= 1 ? (step & 1) : 0;
  auto act_of = [&](int l, int set) { return bfp(set ? t.act_b[l] : t.act[l]); };
  auto act_t_of = [&](int l, int set) { return bfp(set ? t.act_t_b[l] : t.act_t[l]); };
  auto act_in = [&](int l) -> const CUtensorMap& { return ab ? st->act_in_b[l] : st->act_in[l]; };
  auto act_in_t = [&](int l) -> const CUtensorMap& { return ab ? st->act_in_t_b[l] : st->act_in_t[l]; };
  auto act_in_ks = [&](int l) -> const CUtensorMap& { return ab ? st->act_in_ks_b[l] : st->act_in_ks[l]; };
  // Weight gradients of the last two layers beside the remaining dgrad products (their dZ comes
  // out of the fused last-layer kernel): layer L-1 then writes the other of its two bf16 copies,
  // because dgrad through it still reads the current one.
  const bool split_wg = merged && fused_tail && overlap && L >= 3 && st->dbl_layer == L - 1;
  const int rd = st->w16_cur;                                  // copy read in this step
  const int wr = split_wg ? (shared_w ? 0 : 1 - rd) : rd;      // copy written in this step
  auto w_k = [&](int l) -> const CUtensorMap& {
    return (l == st->dbl_layer && rd == 1) ? st->w_b : st->w[l]; };
  auto w_mn = [&](int l) -> const CUtensorMap& {
    return (l == st->dbl_layer && rd == 1) ? st->w_mn_b : st->w_mn[l]; };
  auto w_st = [&](int l) -> const CUtensorMap* {
    return (l == st->dbl_layer && wr == 1) ? &st->w16_st_b : &st->w16_st[l]; };
  const int xb = step & 1;                          // batch buffer of this step
  cudaStream_t main_s = c->stream;
  auto layer_ref = [&](int l) {
    WgradLayerRef r{};
    r.plan = &st->wgrad[l];
    r.dzt = &st->dz_t[l];
    r.at = l == 1 ? &st->x_in_t[xb] : &act_in_t(l);
    r.w32 = &st->w32[l];
    r.w16 = w_st(l);
    r.w32_shared = shared_w ? &st->w32g[l] : nullptr;
    r.u32 = st->wgrad_mom ? &st->u32[l] : nullptr;
    return r;
  };

  cudaError_t e;
#define TC_TRY(call) do { if ((e = (call)) != cudaSuccess) { c->stream = main_s; return e; } } while (0)

  // labels and indices are per step as well: they live beside the batch buffer they belong to
  int32_t* idx_b = idx;
  int32_t* labels_b = labels;
  if (step == 1) st->gathered_step = 0;
  if (st->gathered_step == step) {
    // the launch-by-launch form gathered this step's batch before the previous step's layer-1
    // weight gradient, which read it
  } else if (step == 1 || !overlap) {
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
    const CUtensorMap& wm = shared_w ? st->wg[l] : w_k(l);
    const CUtensorMap& am = l == 1 ? st->x_in[xb] : act_in(l);
    if (l <= done) {
      // A_l of this step came out of the previous step's weight-gradient launch of this layer
    } else if (l < L && shared_w && c->schedule == 0 && st->dense[l].ok) {
      // every learner holds w~: one dense product over the batch rows of all learners
      TC_TRY(launch_fwd_dense(c, st->dense[l], st->wg[l], st->in2d[l][l == 1 ? xb : ab], ly.out,
                              c->buf.global_w + ly.b_off, act_of(l, ab), act_t_of(l, ab)));
    } else if (l < L) {
      g.out_bm = act_of(l, ab); g.out_mb = act_t_of(l, ab);
      if (c->schedule == 0 && st->fwd_ks[l].splits > 1)
        TC_TRY(launch_gemm_ks(c, wm, l == 1 ? st->x_in_ks[xb] : act_in_ks(l), st->fwd_ks[l], g));
      else
        TC_TRY(launch_gemm<EPI_FWD_HIDDEN>(c, MAVG_K_FWD, wm, am, st->fwd[l], g));
    } else if (fused_tail) {
      // last layer forward, loss, dZ_L and dgrad_L in one CUDA-core kernel
      TailLaunch tl{};
      tl.a_bm = L >= 2 ? act_of(L - 1, ab) : bfp(t.xg[xb]);
      tl.w16 = (shared_w ? bfp(t.w16g) : bfp(t.w16)) + t.sh_off[L - 1];
      tl.w16_stride = shared_w ? 0 : t.n16;
      tl.shared_w = shared_w;
      tl.labels = labels_b; tl.loss_out = losses + (step - 1); tl.loss_stride = K;
      tl.dz_t = bfp(t.dz_t[L]);
      if (L >= 2) { tl.dzp_bm = bfp(t.dz[L - 1]); tl.dzp_mb = bfp(t.dz_t[L - 1]); }
      tl.part = (float*)(ws + t.tail_part);
      tl.mom = mom;
      TC_TRY(launch_tail_fused(c, tl));
      // bias steps and loss: beside the backward pass, joined at the end of the step
      if (overlap) {
        TC_TRY(cudaEventRecord(st->ev_fork, main_s));
        TC_TRY(cudaStreamWaitEvent(st->s_wgrad, st->ev_fork, 0));
        c->stream = st->s_wgrad;
        if (split_wg) {
          // the last two layers' weight gradients first (they are on the way of the next
          // step), leaving the SMs of the dgrad tiles alone; then the bias steps and the loss
          WgradLayerRef refs[2] = {layer_ref(L), layer_ref(L - 1)};
          const int busy = cfg.P * st->dgrad[L - 1].m_tiles;
          const int cap = c->sm_count - busy >= 32 ? c->sm_count - busy : 0;
          TC_TRY(launch_wgrad_multi(c, 2, refs, mom, cap));
        }
        TC_TRY(launch_tail_finish(c, tl));
        c->stream = main_s;
        tail_on_side = true;
      } else {
        TC_TRY(launch_tail_finish(c, tl));
      }
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

  bool side_used = tail_on_side;
  for (int l = L; l >= 1; --l) {
    const MlpLayer& ly = c->layers[l - 1];
    if (l > 1 && !(fused_tail && l == L)) {
      const MlpLayer& below = c->layers[l - 2];
      TcArgs g{};
      g.M = ly.in; g.N = B;
      g.a_batched = shared_w ? 0 : 1; g.b_batched = 1;
      g.part = part; g.counters = counters;
      g.bias_rep = c->buf.replicas; g.bias_off = below.b_off;
      g.bias_in = shared_w ? c->buf.global_w : c->buf.replicas;
      g.bias_in_stride = shared_w ? 0 : c->buf.replica_stride;
      g.out_bm = bfp(t.dz[l - 1]); g.out_mb = bfp(t.dz_t[l - 1]);
      g.mask_mb = act_t_of(l - 1, ab);
      g.a_mn = 1;
      g.mom = mom;
      TC_TRY(launch_gemm<EPI_DGRAD>(c, MAVG_K_DGRAD, shared_w ? st->wg_mn[l] : w_mn(l),
                                    st->dz[l], st->dgrad[l], g));
    }
    const CUtensorMap& bm = l == 1 ? st->x_in_t[xb] : act_in_t(l);
    if (merged) continue;        // all layers' weight gradients follow in one launch
    if (l <= ride) continue;     // after the dgrad chain, in ascending order (below)
    if (overlap && l > 1) {
      TC_TRY(cudaEventRecord(st->ev_fork, main_s));
      TC_TRY(cudaStreamWaitEvent(st->s_wgrad, st->ev_fork, 0));
      c->stream = st->s_wgrad;
      TC_TRY(launch_wgrad_stream(c, st->wgrad[l], st->dz_t[l], bm, st->w32[l], *w_st(l),
                                 shared_w ? &st->w32g[l] : nullptr, &st->u32[l], mom));
      c->stream = main_s;
      side_used = true;
    } else {
      TC_TRY(launch_wgrad_stream(c, st->wgrad[l], st->dz_t[l], bm, st->w32[l], *w_st(l),
                                 shared_w ? &st->w32g[l] : nullptr, &st->u32[l], mom));
    }
  }
  // Layers whose launch takes the next step's forward product along: layer l's needs A_{l-1} of
  // the next step, so they run in ascending order, each leaving A_l of the next step behind (in
  // the other set of activation buffers: this step's A_l is still an operand of layer l+1's
  // launch).  Layer 1 reads the next step's gathered
  // batch; only layer 1's bf16 copy has no other reader and is left unwritten.
  for (int l = 1; l <= ride; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    const int nb = (step + 1) & 1;
    if (l == 1) {
      if (overlap) {
        TC_TRY(cudaStreamWaitEvent(main_s, st->ev_gather_done, 0));
      } else {
        TC_TRY(launch_sample_gather(c, round, step + 1, idx_b, labels_b, bfp(t.xg[nb]), bfp(t.xt[nb])));
        st->gathered_step = step + 1;
      }
    }
    const CUtensorMap& bm = l == 1 ? st->x_in_t[xb] : act_in_t(l);
    WgradFwdNext fn{};
    fn.xn = &st->a_next[l][nb];
    fn.zpart = (float*)(ws + t.zpart);
    fn.zcount = (int*)(ws + t.zcount);
    fn.bias_off = ly.b_off;
    fn.out_rows = ly.out;
    fn.out_bm = act_of(l, nb);
    fn.out_mb = act_t_of(l, nb);
    fn.store_w16 = l > 1;
    TC_TRY(launch_wgrad_stream(c, st->wgrad_f[l], st->dz_t[l], bm, st->w32[l], *w_st(l),
                               shared_w ? &st->w32g[l] : nullptr, &st->u32[l], mom, &fn));
    st->fwd_done = l;
  }
  if (merged) {
    // largest layer first, so that the small ones fill the ragged end of the launch
    WgradLayerRef refs[MAVG_MAX_LAYERS];
    const int top = split_wg ? L - 2 : L;      // the last two layers already run on the side
    for (int l = 1; l <= top; ++l) refs[l - 1] = layer_ref(l);
    TC_TRY(launch_wgrad_multi(c, top, refs, mom));
  }
  st->w16_cur = wr;
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
