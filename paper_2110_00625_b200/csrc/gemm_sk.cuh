// Forward (hidden layer) and dgrad products of large workloads as ONE persistent launch that
// keeps every SM streaming weights from the first to the last byte.
//
// The products are  Z^T[M, B] = W[M, K] . A[B, K]^T  per learner, M the 128-row MMA dimension
// (features), the whole batch one N tile.  Work is counted in slabs of 64 contraction elements of
// a 256-row "super tile" (two 128-row MMA tiles that share the batch operand, so that an SM takes
// in the batch tile once per 32 KB of weights instead of once per 16 KB).  The launch has one
// block per SM; block i takes the i-th of equal contiguous ranges of the slab sequence
// (learner-major, then super tile, then slab) -- whatever the number of tiles, every SM streams
// the same number of bytes, and a range crosses tile boundaries without stopping its TMA ring.
// Inside a block: a producer warp fills the ring, one thread issues the MMAs into one of two
// accumulator buffers in tensor memory, eight epilogue warps drain the other one.
//
// A range that begins or ends inside a tile holds only part of that tile's contraction.  Such a
// block writes its fp32 partial tile to scratch memory and adds one to the tile's counter; the
// block whose addition completes the count (whichever it is: nobody waits for anybody) sums the
// partials in ascending order of their position in the contraction and applies the layer's tail.
// The split points depend only on the shapes and on the number of blocks, so the result is the
// same from run to run.  A tile that lies inside one range is finished straight from tensor
// memory.  Tails: bias + ReLU and both orientations of A_l (forward); ReLU mask, dZ in both
// orientations and the bias step of the layer below (dgrad), as in gemm_unit.cuh.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_unit.cuh"
#include "tc_ptx.cuh"

namespace mavg {
namespace gemm {

constexpr int kSkRows = 256;                 // rows of a super tile
constexpr int kSkThreads = 320;              // warp 0 producer, warp 1 MMA, warps 2-9 epilogue
enum { ERR_SK_PRODUCER = 41, ERR_SK_MMA = 42, ERR_SK_EPILOGUE = 43 };

struct SkArgs {
  int M, N;                 // rows of A (features of the output); batch (= N tile, multiple of 16)
  int mt2;                  // super tiles per learner
  int nkb;                  // slabs per tile
  int stages;
  int P;
  long long total;          // P * mt2 * nkb slabs
  int a_batched, a_mn;      // as TcArgs
  uint32_t tmem_cols;       // power of two >= 4 N
  float* part;              // partial tiles: slot s at part + s * N * 256, element [column][row]
  int* tile_ctr;            // one per (learner, super tile); zero between launches
  float* bias_rep; long long bias_off;
  const float* bias_in; long long bias_in_stride;
  __nv_bfloat16* out_bm;    // [P, B, M]
  __nv_bfloat16* out_mb;    // [P, M, B]
  const __nv_bfloat16* mask_mb;   // dgrad: forward activation [P, M, B]
  long long rep_stride;
  float gamma;
  MomArgs mom;
  int* status;
};

struct SkShared {
  uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_slot;
  int abort_flag;
  int last_flag, c_first, c_last;
};

// first slab of block c's range
__device__ __forceinline__ long long sk_start(long long total, int c, int grid) {
  return total * c / grid;
}
// block whose range holds slab x
__device__ __forceinline__ int sk_owner(long long total, long long x, int grid) {
  int c = (int)(x * grid / total);
  while (c + 1 < grid && sk_start(total, c + 1, grid) <= x) ++c;
  while (c > 0 && sk_start(total, c, grid) > x) --c;
  return c;
}

// ORs a predicate over the 256 epilogue threads (barrier 1): a warp that gave up a wait tells the
// others at the next counted barrier, and they all leave together.
__device__ __forceinline__ bool epilogue_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
      "barrier.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

// Tail of one row (feature m of learner p) of a finished tile, eight batch columns at a time;
// load8(cc, z) delivers the accumulator's columns cc..cc+7 of this thread's row.
template <int EPI, typename Load8>
__device__ __forceinline__ void sk_tail_row(const SkArgs& g, int p, int m, bool m_ok, Load8 load8) {
  float* bias = g.bias_rep + (size_t)p * g.rep_stride + g.bias_off;
  const float bias_pre =
      m_ok ? g.bias_in[(size_t)p * g.bias_in_stride + g.bias_off + m] : 0.f;
  const __nv_bfloat16* mrow =
      EPI == EPI_DGRAD ? g.mask_mb + ((size_t)p * g.M + (m_ok ? m : 0)) * g.N : nullptr;
  __nv_bfloat16* orow = g.out_mb + ((size_t)p * g.M + (m_ok ? m : 0)) * g.N;
  float dsum = 0.f;
  uint4 mk = make_uint4(0, 0, 0, 0);
  if (EPI == EPI_DGRAD && m_ok) mk = *reinterpret_cast<const uint4*>(mrow);
#pragma unroll 1
  for (int cc = 0; cc < g.N; cc += 8) {
    float z[8];
    load8(cc, z);
    uint4 mkn = make_uint4(0, 0, 0, 0);                 // next group's mask, in flight meanwhile
    if (EPI == EPI_DGRAD && m_ok && cc + 8 < g.N) mkn = *reinterpret_cast<const uint4*>(mrow + cc + 8);
    const __nv_bfloat16* mh = reinterpret_cast<const __nv_bfloat16*>(&mk);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float v = z[j];
      if (EPI == EPI_DGRAD) {
        v = __bfloat162float(mh[j]) > 0.f ? v : 0.f;    // ReLU'(0) = 0
        dsum += v;
      } else {
        v += bias_pre;
        v = v > 0.f ? v : 0.f;
      }
      z[j] = v;
    }
    uint32_t h4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 h2 = __floats2bfloat162_rn(z[2 * j], z[2 * j + 1]);
      h4[j] = *reinterpret_cast<uint32_t*>(&h2);
    }
    if (m_ok) {
      const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(h4);
      *reinterpret_cast<uint4*>(orow + cc) = make_uint4(h4[0], h4[1], h4[2], h4[3]);
      __nv_bfloat16* dbm = g.out_bm + ((size_t)p * g.N + cc) * g.M + m;
#pragma unroll
      for (int j = 0; j < 8; ++j) dbm[(size_t)j * g.M] = hh[j];
    }
    mk = mkn;
  }
  if (EPI == EPI_DGRAD && m_ok) {
    // bias step of the layer below: b[m] -= gamma * sum_b dZ[b, m], columns added in ascending order
    float* ub = g.mom.u ? g.mom.u + (size_t)p * g.mom.u_stride + g.bias_off + m : nullptr;
    local_update(bias + m, bias_pre, ub, g.mom.read_u, dsum, g.gamma, g.mom.beta);
  }
}

template <int EPI>
__global__ void __launch_bounds__(kSkThreads, 1)
k_tc_gemm_sk(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const SkArgs g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) SkShared sh;
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int BN = g.N;
  const int b_bytes = BN * kBK * 2;
  const int stage_bytes = 2 * kATileBytes + b_bytes;
  const int stages = g.stages;

  grid_launch_dependents();
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < stages; ++s) {
      mbar_init(&sh.full_bar[s], 1);
      mbar_init(&sh.empty_bar[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sh.acc_full[b], 1);
      mbar_init(&sh.acc_empty[b], 8);       // lane 0 of each epilogue warp
    }
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
  grid_dependency_wait();

  const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
  const long long s0 = sk_start(g.total, cta, grid), s1 = sk_start(g.total, cta + 1, grid);
  volatile int* abortp = &sh.abort_flag;
  // next segment of this block's range: slabs [kb0, kb1) of `tile`
  auto next_seg = [&](long long& pos, int& tile, int& kb0, int& kb1) -> bool {
    if (pos >= s1) return false;
    tile = (int)(pos / g.nkb);
    kb0 = (int)(pos - (long long)tile * g.nkb);
    const long long tile_end = (long long)(tile + 1) * g.nkb;
    const long long end = tile_end < s1 ? tile_end : s1;
    kb1 = kb0 + (int)(end - pos);
    pos = end;
    return true;
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0, issued = 0;
      long long pos = s0;
      int tile, kb0, kb1;
      bool ok = true;
      while (ok && next_seg(pos, tile, kb0, kb1)) {
        const int p = tile / g.mt2, m0 = (tile % g.mt2) * kSkRows;
        const int pa = g.a_batched ? p : 0;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % stages;
          if (!mbar_wait(&sh.empty_bar[s], ((it / stages) & 1) ^ 1, abortp, g.status, ERR_SK_PRODUCER)) {
            ok = false;
            break;
          }
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          mbar_arrive_expect_tx(&sh.full_bar[s], (uint32_t)stage_bytes);
          if (g.a_mn) {        // per 128-row tile two 64-wide halves, each 64 K-rows of 128 bytes
#pragma unroll
            for (int h = 0; h < 4; ++h)
              tma_load_3d(sa + h * (kATileBytes / 2), &tmA, &sh.full_bar[s], m0 + 64 * h, kb * kBK, pa);
          } else {
            tma_load_3d(sa, &tmA, &sh.full_bar[s], kb * kBK, m0, pa);
            tma_load_3d(sa + kATileBytes, &tmA, &sh.full_bar[s], kb * kBK, m0 + kBM, pa);
          }
          tma_load_3d(sa + 2 * kATileBytes, &tmB, &sh.full_bar[s], kb * kBK, 0, p);
          issued = it + 1;
        }
      }
      if (*abortp) {
        // give the copies already issued a bounded chance to land before the block retires
        const uint32_t first = issued > (uint32_t)stages ? issued - stages : 0;
        for (uint32_t i = first; i < issued; ++i) {
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(&sh.full_bar[i % stages], (i / stages) & 1))
            if (global_timer_ns() - t0 > wait_limit_ns(g.status)) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, BN, g.a_mn);
      const uint32_t a_step = g.a_mn ? (16 * 128) >> 4 : 2;
      uint32_t it = 0, seg = 0;
      long long pos = s0;
      int tile, kb0, kb1;
      bool ok = true;
      while (ok && next_seg(pos, tile, kb0, kb1)) {
        const int buf = seg & 1;
        if (!mbar_wait(&sh.acc_empty[buf], ((seg >> 1) & 1) ^ 1, abortp, g.status, ERR_SK_MMA)) break;
        tc_fence_after_sync();
        const uint32_t d0 = tmem_base + (uint32_t)(buf * 2 * BN);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % stages;
          if (!mbar_wait(&sh.full_bar[s], (it / stages) & 1, abortp, g.status, ERR_SK_MMA)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
          const uint64_t bdesc = smem_desc_k_sw128(sa + 2 * kATileBytes);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            const uint64_t adesc = g.a_mn ? smem_desc_mn_sw128(sa + sub * kATileBytes)
                                          : smem_desc_k_sw128(sa + sub * kATileBytes);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(d0 + (uint32_t)(sub * BN), adesc + a_step * k, bdesc + 2 * k, idesc,
                        (uint32_t)((kb > kb0) || k != 0));
          }
          umma_commit(&sh.empty_bar[s]);
        }
        if (ok) umma_commit(&sh.acc_full[buf]);
        ++seg;
      }
    }
    __syncwarp();
  } else if (warp < 10) {
    const int ew = warp - 2;
    const int q = warp & 3;                    // TMEM lane quarter this warp may read
    const int sub = ew >> 2;                   // which 128-row tile of the super tile
    const int row = sub * kBM + q * 32 + lane; // row inside the super tile
    uint32_t seg = 0;
    long long pos = s0;
    int tile, kb0, kb1;
    bool failed = false;
    while (next_seg(pos, tile, kb0, kb1)) {
      const int buf = seg & 1;
      if (!failed && !mbar_wait(&sh.acc_full[buf], (seg >> 1) & 1, abortp, g.status, ERR_SK_EPILOGUE))
        failed = true;
      tc_fence_after_sync();
      const int p = tile / g.mt2;
      const int m = (tile % g.mt2) * kSkRows + row;
      const bool m_ok = m < g.M;
      const uint32_t taddr =
          tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * BN + sub * BN);
      const bool whole = kb0 == 0 && kb1 == g.nkb;
      if (whole) {
        if (!failed) {
          sk_tail_row<EPI>(g, p, m, m_ok, [&](int cc, float (&z)[8]) {
            uint32_t r8[8];
            tmem_ld_8cols(taddr + (uint32_t)cc, r8);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j) z[j] = __uint_as_float(r8[j]);
          });
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_one(&sh.acc_empty[buf]);
        }
      } else {
        // part of the tile's contraction: publish it, count, and finish the tile if this was
        // the last part to arrive
        const int slot = 2 * cta + (kb0 == 0 ? 1 : 0);
        if (!failed) {
          float* dst = g.part + (size_t)slot * BN * kSkRows + row;
#pragma unroll 1
          for (int cc = 0; cc < BN; cc += 8) {
            uint32_t r8[8];
            tmem_ld_8cols(taddr + (uint32_t)cc, r8);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[(size_t)(cc + j) * kSkRows] = __uint_as_float(r8[j]);
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_one(&sh.acc_empty[buf]);
        }
        __threadfence();
        if (epilogue_any(failed)) break;       // all eight warps leave together
        if (ew == 0 && lane == 0) {
          const int cf = sk_owner(g.total, (long long)tile * g.nkb, grid);
          const int cl = sk_owner(g.total, (long long)(tile + 1) * g.nkb - 1, grid);
          const int old = atomicAdd(g.tile_ctr + tile, 1);
          const int last = old == cl - cf;
          if (last) g.tile_ctr[tile] = 0;
          __threadfence();
          sh.c_first = cf;
          sh.c_last = cl;
          sh.last_flag = last;
        }
        epilogue_barrier();
        if (sh.last_flag) {
          const int cf = sh.c_first, cl = sh.c_last;
          sk_tail_row<EPI>(g, p, m, m_ok, [&](int cc, float (&z)[8]) {
#pragma unroll
            for (int j = 0; j < 8; ++j) z[j] = 0.f;
#pragma unroll 1
            for (int c = cf; c <= cl; ++c) {   // ascending position in the contraction
              const float* src = g.part + (size_t)(2 * c + (c == cf ? 1 : 0)) * BN * kSkRows +
                                 (size_t)cc * kSkRows + row;
              float t[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) t[j] = __ldcg(src + (size_t)j * kSkRows);
#pragma unroll
              for (int j = 0; j < 8; ++j) z[j] += t[j];
            }
          });
        }
      }
      ++seg;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, g.tmem_cols);
}

}  // namespace gemm
}  // namespace mavg
