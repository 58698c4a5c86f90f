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
#include <cuda.h>

#include "mlp.cuh"
#include "tc_ptx.cuh"
#include "wgrad_tc.cuh"

namespace mavg {
namespace {

using namespace tc;

constexpr int kBM = 128, kBN = 32, kBK = 64;
constexpr int kThreads = 352;   // warp 0 producer, 1 MMA, 2-5 / 6-9 epilogue groups, 10 stores
constexpr int kMaxSlots = 6;
constexpr int kW32Bytes = kBM * kBN * 4;  // 16 KB, rows of 128 bytes, 128-byte swizzle
constexpr int kW16Bytes = kBM * kBN * 2;  //  8 KB, rows of  64 bytes,  64-byte swizzle
enum { ERR_WG_PRODUCER = 21, ERR_WG_MMA = 22, ERR_WG_EPILOGUE = 23, ERR_WG_STORE = 24 };

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, const void* src, int c0, int c1,
                                             int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_store_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Waits until at most `N` of this thread's store groups still have shared memory left to read.
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

struct WgradArgs {
  int w32_in_batched;      // 0: every learner loads the one shared master array (w~)
  int nkb;                 // 64-wide slabs of the batch (contraction)
  int m_tiles, n_tiles;    // 128-row tiles of out, 32-column tiles of in
  int chunk;               // column tiles per work item
  int n_chunks;            // ceil(n_tiles / chunk)
  int items;               // P * m_tiles * n_chunks
  int slots;               // ring depth
  int a_bufs;              // 1 or 2 buffers for the dZ^T tile
  float gamma;
  float beta;              // learner momentum (MOM)
  int read_u;              // 0: the stored u counts as zero and is not loaded
  int* status;
};

template <bool MOM>
__global__ void __launch_bounds__(kThreads)
k_wgrad_sgd_stream(const __grid_constant__ CUtensorMap tm_dzt,   // bf16 [P, out, B]  load
                   const __grid_constant__ CUtensorMap tm_at,    // bf16 [P, in, B]   load
                   const __grid_constant__ CUtensorMap tm_w32,   // fp32 [P, out, in] store
                   const __grid_constant__ CUtensorMap tm_w32_in,  // fp32 masters to load: the same
                                                                   // array, or w~ [1, out, in] at
                                                                   // the first step of a round
                   const __grid_constant__ CUtensorMap tm_w16,   // bf16 [P, out, in] store
                   const __grid_constant__ CUtensorMap tm_u,     // fp32 [P, out, in] u^j, load + store (MOM)
                   const WgradArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots], out_full[kMaxSlots];
  __shared__ __align__(8) uint64_t tmem_full[2], tmem_empty[2];
  __shared__ __align__(8) uint64_t a_full[2], a_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int a_bytes = g.nkb * kBM * kBK * 2;         // dZ^T tile: nkb slabs of 16 KB
  const int b_bytes = g.nkb * kBN * kBK * 2;         // A^T tile:  nkb slabs of 4 KB
  constexpr int kUBytes = MOM ? kW32Bytes : 0;              // the u tile follows the bf16 tile
  constexpr int kBOff = kW32Bytes + kW16Bytes + kUBytes;    // the A^T slabs come last
  const int slot_bytes = kBOff + b_bytes;                   // multiple of 1024
  uint8_t* a_base = smem;
  uint8_t* slot_base = smem + (size_t)g.a_bufs * a_bytes;

  grid_launch_dependents();
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tm_dzt);
    tma_prefetch_desc(&tm_at);
    tma_prefetch_desc(&tm_w32);
    tma_prefetch_desc(&tm_w32_in);
    tma_prefetch_desc(&tm_w16);
    if (MOM) tma_prefetch_desc(&tm_u);
    for (int s = 0; s < g.slots; ++s) {
      mbar_init(&slot_full[s], 1);
      mbar_init(&slot_empty[s], 1);
      mbar_init(&out_full[s], 4);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tmem_full[b], 1);
      mbar_init(&tmem_empty[b], 4);
      mbar_init(&a_full[b], 1);
      mbar_init(&a_empty[b], 1);
    }
    abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, 64);            // two accumulators of 32 columns
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abortp = &abort_flag;
  grid_dependency_wait();

  // work item -> (learner p, row tile, first column tile, number of column tiles)
  auto decode = [&](int item, int& p, int& m0, int& nt0, int& nt) {
    const int nc = item % g.n_chunks;
    const int rest = item / g.n_chunks;
    const int mt = rest % g.m_tiles;
    p = rest / g.m_tiles;
    m0 = mt * kBM;
    nt0 = nc * g.chunk;
    nt = min(g.chunk, g.n_tiles - nt0);
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t tile_ctr = 0, item_ctr = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < g.items && ok; item += gridDim.x, ++item_ctr) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        const int ab = item_ctr % g.a_bufs;
        const uint32_t a_use = item_ctr / g.a_bufs;
        if (!mbar_wait(&a_empty[ab], (a_use & 1) ^ 1, abortp, g.status, ERR_WG_PRODUCER)) break;
        mbar_arrive_expect_tx(&a_full[ab], (uint32_t)a_bytes);
        for (int kb = 0; kb < g.nkb; ++kb)
          tma_load_3d(a_base + (size_t)ab * a_bytes + (size_t)kb * (kBM * kBK * 2), &tm_dzt,
                      &a_full[ab], kb * kBK, m0, p);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          if (!mbar_wait(&slot_empty[s], (use & 1) ^ 1, abortp, g.status, ERR_WG_PRODUCER)) {
            ok = false;
            break;
          }
          uint8_t* sl = slot_base + (size_t)s * slot_bytes;
          const int i0 = (nt0 + j) * kBN;
          const bool load_u = MOM && g.read_u;
          mbar_arrive_expect_tx(&slot_full[s],
                                (uint32_t)(kW32Bytes + b_bytes + (load_u ? kUBytes : 0)));
          tma_load_3d(sl, &tm_w32_in, &slot_full[s], i0, m0, g.w32_in_batched ? p : 0);
          if (load_u) tma_load_3d(sl + kW32Bytes + kW16Bytes, &tm_u, &slot_full[s], i0, m0, p);
          for (int kb = 0; kb < g.nkb; ++kb)
            tma_load_3d(sl + kBOff + (size_t)kb * (kBN * kBK * 2),
                        &tm_at, &slot_full[s], kb * kBK, i0, p);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, kBN);
      uint32_t tile_ctr = 0, item_ctr = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < g.items && ok; item += gridDim.x, ++item_ctr) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        const int ab = item_ctr % g.a_bufs;
        const uint32_t a_use = item_ctr / g.a_bufs;
        if (!mbar_wait(&a_full[ab], a_use & 1, abortp, g.status, ERR_WG_MMA)) break;
        const uint32_t a_addr = smem_u32(a_base + (size_t)ab * a_bytes);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          const int tb = tile_ctr & 1;
          const uint32_t tuse = tile_ctr >> 1;
          if (!mbar_wait(&slot_full[s], use & 1, abortp, g.status, ERR_WG_MMA) ||
              !mbar_wait(&tmem_empty[tb], (tuse & 1) ^ 1, abortp, g.status, ERR_WG_MMA)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t b_addr = smem_u32(slot_base + (size_t)s * slot_bytes + kBOff);
          for (int kb = 0; kb < g.nkb; ++kb) {
            const uint64_t adesc = smem_desc_k_sw128(a_addr + kb * (kBM * kBK * 2));
            const uint64_t bdesc = smem_desc_k_sw128(b_addr + kb * (kBN * kBK * 2));
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(tmem_base + tb * kBN, adesc + 2 * k, bdesc + 2 * k, idesc,
                        (uint32_t)((kb | k) != 0));
          }
          umma_commit(&tmem_full[tb]);
        }
        if (ok) umma_commit(&a_empty[ab]);     // all MMAs that read this dZ^T tile have finished
      }
    }
    __syncwarp();
  } else if (warp < 10) {
    const int grp = (warp - 2) >> 2;           // epilogue group = TMEM buffer = tile parity
    const int q = warp & 3;                    // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;               // weight row inside the tile
    uint32_t tile_ctr = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < g.items && ok; item += gridDim.x) {
      int p, m0, nt0, nt;
      decode(item, p, m0, nt0, nt);
      for (int j = 0; j < nt; ++j, ++tile_ctr) {
        if ((int)(tile_ctr & 1) != grp) continue;
        const int s = tile_ctr % g.slots;
        const uint32_t use = tile_ctr / g.slots;
        const uint32_t tuse = tile_ctr >> 1;
        // the master tile landed with the same barrier the MMA waited on; the accumulator next
        if (!mbar_wait(&slot_full[s], use & 1, abortp, g.status, ERR_WG_EPILOGUE) ||
            !mbar_wait(&tmem_full[grp], tuse & 1, abortp, g.status, ERR_WG_EPILOGUE)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        uint32_t acc[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(grp * kBN), acc);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty[grp]);    // this warp is done with the buffer

        uint8_t* sl = slot_base + (size_t)s * slot_bytes;
        uint8_t* w32 = sl + (size_t)r * 128;             // 8 chunks of 16 B, chunk c at c ^ (r & 7)
        uint8_t* w16 = sl + kW32Bytes + (size_t)r * 64;  // 4 chunks, chunk c at c ^ ((r >> 1) & 3)
        uint32_t hp[16];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float4* cell = reinterpret_cast<float4*>(w32 + ((c ^ (r & 7)) << 4));
          float4 w = *cell;
          if (MOM) {
            // the u tile has the master tile's shape and swizzle
            float4* ucell = reinterpret_cast<float4*>(w32 + kW32Bytes + kW16Bytes +
                                                      ((c ^ (r & 7)) << 4));
            float4 u = g.read_u ? *ucell : make_float4(0.f, 0.f, 0.f, 0.f);
            msgd(w.x, u.x, __uint_as_float(acc[4 * c + 0]), g.gamma, g.beta);
            msgd(w.y, u.y, __uint_as_float(acc[4 * c + 1]), g.gamma, g.beta);
            msgd(w.z, u.z, __uint_as_float(acc[4 * c + 2]), g.gamma, g.beta);
            msgd(w.w, u.w, __uint_as_float(acc[4 * c + 3]), g.gamma, g.beta);
            *ucell = u;
          } else {
            w.x = fmaf(-g.gamma, __uint_as_float(acc[4 * c + 0]), w.x);
            w.y = fmaf(-g.gamma, __uint_as_float(acc[4 * c + 1]), w.y);
            w.z = fmaf(-g.gamma, __uint_as_float(acc[4 * c + 2]), w.z);
            w.w = fmaf(-g.gamma, __uint_as_float(acc[4 * c + 3]), w.w);
          }
          *cell = w;
          __nv_bfloat162 h0 = __floats2bfloat162_rn(w.x, w.y);
          __nv_bfloat162 h1 = __floats2bfloat162_rn(w.z, w.w);
          hp[2 * c] = *reinterpret_cast<uint32_t*>(&h0);
          hp[2 * c + 1] = *reinterpret_cast<uint32_t*>(&h1);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
          *reinterpret_cast<uint4*>(w16 + ((c ^ ((r >> 1) & 3)) << 4)) =
              make_uint4(hp[4 * c], hp[4 * c + 1], hp[4 * c + 2], hp[4 * c + 3]);
        fence_proxy_async();                   // generic-proxy writes -> visible to the TMA stores
        __syncwarp();
        if (lane == 0) mbar_arrive(&out_full[s]);
      }
    }
  } else {
    if (lane == 0) {
      uint32_t tile_ctr = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < g.items && ok; item += gridDim.x) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          if (!mbar_wait(&out_full[s], use & 1, abortp, g.status, ERR_WG_STORE)) {
            ok = false;
            break;
          }
          uint8_t* sl = slot_base + (size_t)s * slot_bytes;
          const int i0 = (nt0 + j) * kBN;
          tma_store_3d(&tm_w32, sl, i0, m0, p);
          tma_store_3d(&tm_w16, sl + kW32Bytes, i0, m0, p);
          if (MOM) tma_store_3d(&tm_u, sl + kW32Bytes + kW16Bytes, i0, m0, p);
          tma_store_commit();
          // the slot of the previous tile is free once its stores have read shared memory
          if (tile_ctr > 0) {
            tma_store_wait_read<1>();
            mbar_arrive(&slot_empty[(tile_ctr - 1) % g.slots]);
          }
        }
      }
      tma_store_wait_read<0>();
      if (tile_ctr > 0 && ok) mbar_arrive(&slot_empty[(tile_ctr - 1) % g.slots]);
    }
    __syncwarp();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 64);
}

}  // namespace

WgradPlan plan_wgrad_stream(int out, int in, int B, int P, int sm_count, bool momentum) {
  WgradPlan w{};
  w.nkb = (B + kBK - 1) / kBK;
  w.m_tiles = (out + kBM - 1) / kBM;
  w.n_tiles = (in + kBN - 1) / kBN;
  const long total = (long)P * w.m_tiles * w.n_tiles;
  long chunk = total / (8L * sm_count);
  if (chunk < 1) chunk = 1;
  if (chunk > 16) chunk = 16;
  if (chunk > w.n_tiles) chunk = w.n_tiles;
  w.chunk = (int)chunk;
  w.n_chunks = (w.n_tiles + w.chunk - 1) / w.chunk;
  w.items = P * w.m_tiles * w.n_chunks;
  const int a_bytes = w.nkb * kBM * kBK * 2;
  const int slot_bytes = kW32Bytes + kW16Bytes + (momentum ? kW32Bytes : 0) + w.nkb * kBN * kBK * 2;
  const int budget = 220 * 1024;
  w.a_bufs = 2;
  w.slots = (budget - 2 * a_bytes) / slot_bytes;
  if (w.slots < 2) {
    w.a_bufs = 1;
    w.slots = (budget - a_bytes) / slot_bytes;
  }
  if (w.slots > kMaxSlots) w.slots = kMaxSlots;
  w.smem = (size_t)w.a_bufs * a_bytes + (size_t)w.slots * slot_bytes + 1024;
  w.grid = w.items < sm_count ? w.items : sm_count;
  return w;
}

cudaError_t wgrad_stream_prepare() {
  cudaError_t e = cudaFuncSetAttribute(k_wgrad_sgd_stream<false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_wgrad_sgd_stream<true>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
}

cudaError_t launch_wgrad_stream(mavg_ctx* c, const WgradPlan& w, const CUtensorMap& dzt,
                                const CUtensorMap& at, const CUtensorMap& w32,
                                const CUtensorMap& w16, const CUtensorMap* w32_shared,
                                const CUtensorMap* u32, const MomArgs& mom) {
  WgradArgs g{};
  g.w32_in_batched = w32_shared ? 0 : 1;
  g.nkb = w.nkb;
  g.m_tiles = w.m_tiles;
  g.n_tiles = w.n_tiles;
  g.chunk = w.chunk;
  g.n_chunks = w.n_chunks;
  g.items = w.items;
  g.slots = w.slots;
  g.a_bufs = w.a_bufs;
  g.gamma = c->cfg.local_lr;
  g.beta = mom.beta;
  g.read_u = mom.read_u;
  g.status = (int*)ws_ptr(c, c->ws.status);
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)w.grid);
  lc.blockDim = dim3(kThreads);
  lc.dynamicSmemBytes = w.smem;
  lc.stream = c->stream;
  cudaLaunchAttribute at_[1];
  at_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at_[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at_;
  lc.numAttrs = 1;
  prof_begin(c, MAVG_K_WGRAD_SGD);
  cudaError_t e = (mom.u && u32)
      ? cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<true>, dzt, at, w32,
                           w32_shared ? *w32_shared : w32, w16, *u32, g)
      : cudaLaunchKernelEx(&lc, k_wgrad_sgd_stream<false>, dzt, at, w32,
                           w32_shared ? *w32_shared : w32, w16, w32, g);
  prof_end(c);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace mavg
