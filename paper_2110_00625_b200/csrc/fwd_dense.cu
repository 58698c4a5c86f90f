// Dense first-step forward product of a hidden layer (see fwd_dense.cuh): one 128 x 256 output
// tile per block, operands staged by TMA in a ring of 48 KB stages (16 KB of w~ rows, 32 KB of
// batch rows of four or more learners), tcgen05.mma with a 128 x 256 fp32 accumulator in tensor
// memory, bias + ReLU + bf16 in the epilogue, written in both orientations.
#include <cuda.h>

#include <algorithm>

#include "fwd_dense.cuh"
#include "gemm_unit.cuh"
#include "tc_ptx.cuh"

namespace mavg {
namespace {

using namespace tc;
using namespace gemm;

constexpr int kDenseThreads = 320;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
constexpr int kDenseStageBytes = kATileBytes + kDenseCols * kBK * 2;
constexpr int kDenseMaxStages = 4;

struct DenseArgs {
  int M;          // rows of the layer (out)
  int NB;         // P * B: batch rows of all learners
  int B;
  int nkb, stages, n_tiles;
  const float* bias;
  __nv_bfloat16* out_bm;   // [P, B, M] = [NB, M]
  __nv_bfloat16* out_mb;   // [P, M, B]
  int* status;
};

__global__ void __launch_bounds__(kDenseThreads, 1)
k_fwd_dense(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
            const DenseArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) GemmShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  grid_launch_dependents();
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmX);
    gemm_init_barriers(sh, g.stages);
    sh.abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&sh.tmem_slot, kDenseCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh.tmem_slot;
  grid_dependency_wait();

  const int n_tile = (int)blockIdx.x % g.n_tiles, m_tile = (int)blockIdx.x / g.n_tiles;
  const int m0 = m_tile * kBM, n0 = n_tile * kDenseCols;
  const int stages = g.stages;
  volatile int* abortp = &sh.abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int i = 0; i < g.nkb; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&sh.empty_bar[s], (u & 1) ^ 1, abortp, g.status, ERR_PRODUCER)) break;
        uint8_t* sa = smem + (size_t)s * kDenseStageBytes;
        mbar_arrive_expect_tx(&sh.full_bar[s], (uint32_t)kDenseStageBytes);
        tma_load_3d(sa, &tmW, &sh.full_bar[s], i * kBK, m0, 0);
        tma_load_3d(sa + kATileBytes, &tmX, &sh.full_bar[s], i * kBK, n0, 0);
        issued = i + 1;
      }
      if (*abortp) {
        // give the copies already issued a bounded chance to land before the block retires
        for (int i = max(0, issued - stages); i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&sh.full_bar[i % stages], (i / stages) & 1))
            if (global_timer_ns() - t0 > wait_limit_ns(g.status)) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, kDenseCols);
      bool ok = true;
      for (int i = 0; i < g.nkb; ++i) {
        const int s = i % stages, u = i / stages;
        if (!mbar_wait(&sh.full_bar[s], u & 1, abortp, g.status, ERR_MMA)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t sa = smem_u32(smem + (size_t)s * kDenseStageBytes);
        const uint64_t adesc = smem_desc_k_sw128(sa);
        const uint64_t bdesc = smem_desc_k_sw128(sa + kATileBytes);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)
          umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (uint32_t)((i | k) != 0));
        umma_commit(&sh.empty_bar[s]);
      }
      if (ok) umma_commit(&sh.acc_bar);
    }
    __syncwarp();
  } else {
    // warp (q, half): TMEM lanes [32q, 32q + 32) (the lanes a warp with index mod 4 == q may
    // read) and every second 32-column chunk; one weight row per lane
    const int q = warp & 3, half = (warp - 2) >> 2;
    const int m = m0 + q * 32 + lane;
    const bool m_ok = m < g.M;
    const float bias = m_ok ? g.bias[m] : 0.f;
    if (mbar_wait(&sh.acc_bar, 0, abortp, g.status, ERR_EPILOGUE)) {
      tc_fence_after_sync();
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
      for (int c0 = half * 32; c0 < kDenseCols; c0 += 64) {
        float z[32];
        load_acc_chunk(lane_addr, c0, kDenseCols, z);
        if (!m_ok) continue;
        // the batch is a multiple of 16: a group of eight columns belongs to one learner
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int n = n0 + c0 + 8 * v;
          if (n >= g.NB) break;
          const int p = n / g.B, b = n - p * g.B;
          uint32_t h4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float a0 = z[8 * v + 2 * j] + bias, a1 = z[8 * v + 2 * j + 1] + bias;
            __nv_bfloat162 h2 = __floats2bfloat162_rn(a0 > 0.f ? a0 : 0.f, a1 > 0.f ? a1 : 0.f);
            h4[j] = *reinterpret_cast<uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(g.out_mb + ((size_t)p * g.M + m) * g.B + b) =
              make_uint4(h4[0], h4[1], h4[2], h4[3]);
          const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(h4);
          __nv_bfloat16* dbm = g.out_bm + (size_t)n * g.M + m;
#pragma unroll
          for (int j = 0; j < 8; ++j) dbm[(size_t)j * g.M] = hh[j];
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kDenseCols);
}

}  // namespace

DensePlan plan_fwd_dense(int out, int in, int B, int P, int sm_count) {
  DensePlan pl{};
  pl.m_tiles = (out + kBM - 1) / kBM;
  pl.n_tiles = (int)(((long)P * B + kDenseCols - 1) / kDenseCols);
  pl.nkb = (in + kBK - 1) / kBK;
  pl.stages = std::min(kDenseMaxStages, pl.nkb);
  pl.smem = (size_t)pl.stages * kDenseStageBytes + 1024;
  // the box of the batch operand must fit the array, and a third of the SMs must get a tile:
  // below that the per-learner tiles, of which there are P per row tile, keep more SMs busy
  pl.ok = (long)P * B >= kDenseCols && out >= kBM && (long)pl.m_tiles * pl.n_tiles * 3 >= sm_count;
  return pl;
}

cudaError_t fwd_dense_prepare() {
  return cudaFuncSetAttribute(k_fwd_dense, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kDenseMaxStages * kDenseStageBytes + 1024);
}

cudaError_t launch_fwd_dense(mavg_ctx* c, const DensePlan& pl, const CUtensorMap& w,
                             const CUtensorMap& x, int out, const float* bias,
                             __nv_bfloat16* out_bm, __nv_bfloat16* out_mb) {
  DenseArgs g{};
  g.M = out;
  g.NB = c->cfg.P * c->cfg.B;
  g.B = c->cfg.B;
  g.nkb = pl.nkb;
  g.stages = pl.stages;
  g.n_tiles = pl.n_tiles;
  g.bias = bias;
  g.out_bm = out_bm;
  g.out_mb = out_mb;
  g.status = (int*)ws_ptr(c, c->ws.status);
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)(pl.m_tiles * pl.n_tiles));
  lc.blockDim = dim3(kDenseThreads);
  lc.dynamicSmemBytes = pl.smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  prof_begin(c, MAVG_K_FWD);
  cudaError_t e = cudaLaunchKernelEx(&lc, k_fwd_dense, w, x, g);
  prof_end(c);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace mavg
