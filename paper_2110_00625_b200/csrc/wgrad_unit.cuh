// Roles of the streaming weight-gradient + SGD block (see wgrad_tc.cu for the scheme), used by its
// one-layer and its several-layers kernel.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace mavg {
namespace wgrad {

using namespace tc;

constexpr int kBM = 128, kBN = 32, kBK = 64;
constexpr int kThreads = 352;      // warp 0 producer, 1 MMA, 2-5 / 6-9 epilogue groups, 10 stores
constexpr int kThreadsFwd = 512;   // + warp 11 forward MMAs, 12-15 forward accumulator (fwd_next)
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
__device__ __forceinline__ void tma_store_3d_hint(const CUtensorMap* m, const void* src, int c0,
                                                  int c1, int c2, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group.L2::cache_hint"
      " [%0, {%2, %3, %4}], [%1], %5;"
      ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "l"(pol)
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
  int items;               // whole_rows + (P * m_tiles - whole_rows) * n_chunks
  int whole_rows;          // the first whole_rows (learner, row tile) pairs are one work item each:
                           // all n_tiles column tiles in one run; the others are cut into
                           // n_chunks runs of chunk tiles (0 everywhere but in plans that balance
                           // a riding forward product's long runs over the blocks)
  int slots;               // ring depth
  int a_bufs;              // 1 or 2 buffers for the dZ^T tile
  int w16_on_b;            // 1: the bf16 output tile is written over the slot's A^T slabs
  int keep_w32;            // 1: master tiles are loaded and stored with the L2 evict-last hint
                           //    (all learners' masters together fit in half the L2: they are
                           //    read again one step later and should not go through HBM)
  float gamma;
  float beta;              // learner momentum (MOM)
  int read_u;              // 0: the stored u counts as zero and is not loaded
  // Next step's forward product of the same layer, taken from the freshly updated tiles while
  // they are in shared memory (see wgrad_tc.cu): fwd_next = 1 adds, per tile,
  //   Z^T[128 rows, B] += W16_tile[128, 32] . Xn[B, 32]^T
  // into a third TMEM accumulator; per work item the fp32 partial sum goes to
  //   zpart[((p * m_tiles + row tile) * n_chunks + chunk) * B * 128 + b * 128 + row]
  // (not with a single run per row: then the accumulator is the whole product).
  int fwd_next;
  int store_w16;           // 0: the bf16 tile is not written to global memory
  int xn_bytes;            // room in a slot for the next step's input tile [B, 32] bf16 (loaded
                           // only with fwd_next; part of the slot's size whenever the plan has it)
  int batch;               // B
  float* zpart;
  // the work item that completes a row tile's product last adds the partial sums up in ascending
  // run order, adds the bias, applies ReLU and writes A_l of the next step as bf16 in both
  // orientations (out_bm [P, B, out], out_mb [P, out, B]); zcount: one arrival counter per
  // (learner, row tile), zero before and after the launch
  int* zcount;
  const float* bias_rep;   // masters [P, rep_stride]; the layer's bias at bias_off
  int64_t rep_stride, bias_off;
  int out_rows;            // rows of the layer (the last row tile may be ragged)
  __nv_bfloat16* out_bm;
  __nv_bfloat16* out_mb;
  int* status;
};


struct WgradShared {
  uint64_t slot_full[kMaxSlots], slot_empty[kMaxSlots], out_full[kMaxSlots];
  uint64_t tmem_full[2], tmem_empty[2];
  uint64_t a_full[2], a_empty[2];
  uint64_t z_done[kMaxSlots];   // the forward MMAs that read this slot's bf16 tile have finished
  uint64_t z_full, z_empty;     // the item's forward accumulator is complete / has been read
  uint64_t z_part, z_flag;      // the item's partial sum is in global memory / z_last is set
  int z_last;                   // this item completed its row tile's product last
  uint32_t tmem_slot;
  int abort_flag;
};

__device__ __forceinline__ void wgrad_init_barriers(WgradShared& sh, int slots) {
  for (int s = 0; s < slots; ++s) {
    mbar_init(&sh.slot_full[s], 1);
    mbar_init(&sh.slot_empty[s], 1);
    mbar_init(&sh.out_full[s], 4);
    mbar_init(&sh.z_done[s], 1);
  }
  mbar_init(&sh.z_full, 1);
  mbar_init(&sh.z_empty, 4);
  mbar_init(&sh.z_part, 4);
  mbar_init(&sh.z_flag, 1);
  for (int b = 0; b < 2; ++b) {
    mbar_init(&sh.tmem_full[b], 1);
    mbar_init(&sh.tmem_empty[b], 4);
    mbar_init(&sh.a_full[b], 1);
    mbar_init(&sh.a_empty[b], 1);
  }
}

// Tiles and items of the run (vblock, vgrid) of the launch g: what a later run of the same block
// adds to tile_base and item_base.
__device__ __forceinline__ void wgrad_run_totals(const WgradArgs& g, int vblock, int vgrid,
                                                 uint32_t& tiles, uint32_t& items) {
  for (int item = vblock; item < g.items; item += vgrid) {
    const int nt0 = ((item - g.whole_rows) % g.n_chunks) * g.chunk;
    tiles += (uint32_t)(item < g.whole_rows ? g.n_tiles : min(g.chunk, g.n_tiles - nt0));
    items += 1;
  }
}

// Work items vblock, vblock + vgrid, ... of the launch described by g.  Barriers initialised
// (phase 0) and a block-wide barrier passed before; 64 columns of tensor memory at tmem_base.
// A block that makes several runs keeps using the same barriers (g.slots and g.a_bufs must not
// change): tile_base and item_base are the tiles and items of its earlier runs, see
// wgrad_run_totals.
// FWD = false compiles the roles of the riding forward product out (g.fwd_next must be 0).
template <bool MOM, bool FWD>
__device__ __forceinline__ void wgrad_run(const CUtensorMap& tm_dzt, const CUtensorMap& tm_at,
                                          const CUtensorMap& tm_w32, const CUtensorMap& tm_w32_in,
                                          const CUtensorMap& tm_w16, const CUtensorMap& tm_u,
                                          const CUtensorMap& tm_xn,
                                          const WgradArgs& g, int vblock, int vgrid, uint8_t* smem,
                                          WgradShared& sh, uint32_t tmem_base,
                                          uint32_t tile_base = 0, uint32_t item_base = 0) {
  const bool fwd_next = FWD && g.fwd_next != 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int a_bytes = g.nkb * kBM * kBK * 2;         // dZ^T tile: nkb slabs of 16 KB
  const int b_bytes = g.nkb * kBN * kBK * 2;         // A^T tile:  nkb slabs of 4 KB
  // Slot: [master tile 16 KB][u tile 16 KB (MOM)][bf16 tile 8 KB][A^T slabs], or, when the A^T
  // slabs are at least as large as the bf16 tile (g.w16_on_b), without a region of its own for the
  // bf16 tile: the MMA has finished reading A^T when the epilogue writes, so the bf16 tile goes
  // on top of it and more slots fit.
  constexpr int kUBytes = MOM ? kW32Bytes : 0;
  const int w16_off = kW32Bytes + kUBytes;
  const int b_off = g.w16_on_b ? w16_off : w16_off + kW16Bytes;
  const int xn_off = b_off + b_bytes;                       // next step's input tile (fwd_next)
  const int slot_bytes = xn_off + g.xn_bytes;               // multiple of 1024
  constexpr uint32_t kZCol = 2 * kBN;                       // forward accumulator: B columns from here
  uint8_t* a_base = smem;
  uint8_t* slot_base = smem + (size_t)g.a_bufs * a_bytes;
  volatile int* abortp = &sh.abort_flag;

  // work item -> (learner p, row tile, first column tile, number of column tiles)
  auto decode = [&](int item, int& p, int& m0, int& nt0, int& nt) {
    int row;                       // (learner, row tile) pair
    if (item < g.whole_rows) {
      row = item;
      nt0 = 0;
      nt = g.n_tiles;
    } else {
      const int idx = item - g.whole_rows;
      row = g.whole_rows + idx / g.n_chunks;
      nt0 = (idx % g.n_chunks) * g.chunk;
      nt = min(g.chunk, g.n_tiles - nt0);
    }
    const int mt = row % g.m_tiles;
    p = row / g.m_tiles;
    m0 = mt * kBM;
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t tile_ctr = tile_base, item_ctr = item_base;
      bool ok = true;
      const uint64_t pol = l2_policy(g.keep_w32 != 0);
      for (int item = vblock; item < g.items && ok; item += vgrid, ++item_ctr) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        const int ab = item_ctr % g.a_bufs;
        const uint32_t a_use = item_ctr / g.a_bufs;
        if (!mbar_wait(&sh.a_empty[ab], (a_use & 1) ^ 1, abortp, g.status, ERR_WG_PRODUCER)) break;
        mbar_arrive_expect_tx(&sh.a_full[ab], (uint32_t)a_bytes);
        for (int kb = 0; kb < g.nkb; ++kb)
          tma_load_3d(a_base + (size_t)ab * a_bytes + (size_t)kb * (kBM * kBK * 2), &tm_dzt,
                      &sh.a_full[ab], kb * kBK, m0, p);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          if (!mbar_wait(&sh.slot_empty[s], (use & 1) ^ 1, abortp, g.status, ERR_WG_PRODUCER)) {
            ok = false;
            break;
          }
          uint8_t* sl = slot_base + (size_t)s * slot_bytes;
          const int i0 = (nt0 + j) * kBN;
          const bool load_u = MOM && g.read_u;
          mbar_arrive_expect_tx(&sh.slot_full[s],
                                (uint32_t)(kW32Bytes + b_bytes + (load_u ? kUBytes : 0) +
                                           (fwd_next ? g.xn_bytes : 0)));
          if (fwd_next) tma_load_3d(sl + xn_off, &tm_xn, &sh.slot_full[s], i0, 0, p);
          tma_load_3d_hint(sl, &tm_w32_in, &sh.slot_full[s], i0, m0, g.w32_in_batched ? p : 0, pol);
          if (load_u) tma_load_3d(sl + kW32Bytes, &tm_u, &sh.slot_full[s], i0, m0, p);
          for (int kb = 0; kb < g.nkb; ++kb)
            tma_load_3d(sl + b_off + (size_t)kb * (kBN * kBK * 2),
                        &tm_at, &sh.slot_full[s], kb * kBK, i0, p);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(kBM, kBN);
      uint32_t tile_ctr = tile_base, item_ctr = item_base;
      bool ok = true;
      for (int item = vblock; item < g.items && ok; item += vgrid, ++item_ctr) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        const int ab = item_ctr % g.a_bufs;
        const uint32_t a_use = item_ctr / g.a_bufs;
        if (!mbar_wait(&sh.a_full[ab], a_use & 1, abortp, g.status, ERR_WG_MMA)) break;
        const uint32_t a_addr = smem_u32(a_base + (size_t)ab * a_bytes);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          const int tb = tile_ctr & 1;
          const uint32_t tuse = tile_ctr >> 1;
          if (!mbar_wait(&sh.slot_full[s], use & 1, abortp, g.status, ERR_WG_MMA) ||
              !mbar_wait(&sh.tmem_empty[tb], (tuse & 1) ^ 1, abortp, g.status, ERR_WG_MMA)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t b_addr = smem_u32(slot_base + (size_t)s * slot_bytes + b_off);
          for (int kb = 0; kb < g.nkb; ++kb) {
            const uint64_t adesc = smem_desc_k_sw128(a_addr + kb * (kBM * kBK * 2));
            const uint64_t bdesc = smem_desc_k_sw128(b_addr + kb * (kBN * kBK * 2));
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)
              umma_bf16(tmem_base + tb * kBN, adesc + 2 * k, bdesc + 2 * k, idesc,
                        (uint32_t)((kb | k) != 0));
          }
          umma_commit(&sh.tmem_full[tb]);
        }
        if (ok) umma_commit(&sh.a_empty[ab]);     // all MMAs that read this dZ^T tile have finished
      }
    }
    __syncwarp();
  } else if (warp < 10) {
    const int grp = (warp - 2) >> 2;           // epilogue group = TMEM buffer = tile parity
    const int q = warp & 3;                    // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;               // weight row inside the tile
    uint32_t tile_ctr = tile_base;
    bool ok = true;
    for (int item = vblock; item < g.items && ok; item += vgrid) {
      int p, m0, nt0, nt;
      decode(item, p, m0, nt0, nt);
      for (int j = 0; j < nt; ++j, ++tile_ctr) {
        if ((int)(tile_ctr & 1) != grp) continue;
        const int s = tile_ctr % g.slots;
        const uint32_t use = tile_ctr / g.slots;
        const uint32_t tuse = tile_ctr >> 1;
        // the master tile landed with the same barrier the MMA waited on; the accumulator next
        if (!mbar_wait(&sh.slot_full[s], use & 1, abortp, g.status, ERR_WG_EPILOGUE) ||
            !mbar_wait(&sh.tmem_full[grp], tuse & 1, abortp, g.status, ERR_WG_EPILOGUE)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        uint32_t acc[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(grp * kBN), acc);
        tmem_ld_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tmem_empty[grp]);    // this warp is done with the buffer

        uint8_t* sl = slot_base + (size_t)s * slot_bytes;
        uint8_t* w32 = sl + (size_t)r * 128;             // 8 chunks of 16 B, chunk c at c ^ (r & 7)
        uint8_t* w16 = sl + w16_off + (size_t)r * 64;    // 4 chunks, chunk c at c ^ ((r >> 1) & 3)
        uint32_t hp[16];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float4* cell = reinterpret_cast<float4*>(w32 + ((c ^ (r & 7)) << 4));
          float4 w = *cell;
          if (MOM) {
            // the u tile has the master tile's shape and swizzle
            float4* ucell = reinterpret_cast<float4*>(w32 + kW32Bytes + ((c ^ (r & 7)) << 4));
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
        __syncwarp();                          // (and to the forward MMAs, fwd_next)
        if (lane == 0) mbar_arrive(&sh.out_full[s]);
      }
    }
  } else if (warp == 10) {
    if (lane == 0) {
      uint32_t tile_ctr = tile_base;
      bool ok = true;
      int held = -1;          // slot whose stores are committed but not yet known to be read
      uint32_t held_use = 0;
      const uint64_t pol = l2_policy(g.keep_w32 != 0);
      for (int item = vblock; item < g.items && ok; item += vgrid) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          const uint32_t use = tile_ctr / g.slots;
          if (!mbar_wait(&sh.out_full[s], use & 1, abortp, g.status, ERR_WG_STORE)) {
            ok = false;
            break;
          }
          uint8_t* sl = slot_base + (size_t)s * slot_bytes;
          const int i0 = (nt0 + j) * kBN;
          tma_store_3d_hint(&tm_w32, sl, i0, m0, p, pol);
          if (g.store_w16) tma_store_3d(&tm_w16, sl + w16_off, i0, m0, p);
          if (MOM) tma_store_3d(&tm_u, sl + kW32Bytes, i0, m0, p);
          tma_store_commit();
          // A slot is free once its stores have read shared memory.  If the next tile is already
          // waiting to be stored, its stores go out first and this slot is handed back behind
          // them; if not, this thread has nothing else to do, waits for the read here and hands
          // the slot back a whole tile period earlier.
          // (with fwd_next a slot is also still being read by its forward MMAs: z_done)
          if (held >= 0) {
            tma_store_wait_read<1>();
            if (fwd_next && !mbar_wait(&sh.z_done[held], held_use & 1, abortp, g.status, ERR_WG_STORE)) {
              ok = false;
              break;
            }
            mbar_arrive(&sh.slot_empty[held]);
            held = -1;
          }
          {
            const uint32_t nx = tile_ctr + 1;
            if (mbar_try_wait(&sh.out_full[nx % g.slots], (nx / g.slots) & 1)) {
              held = s;
              held_use = use;
            } else {
              tma_store_wait_read<0>();
              if (fwd_next && !mbar_wait(&sh.z_done[s], use & 1, abortp, g.status, ERR_WG_STORE)) {
                ok = false;
                break;
              }
              mbar_arrive(&sh.slot_empty[s]);
            }
          }
        }
      }
      if (held >= 0) {
        tma_store_wait_read<0>();
        if (!fwd_next || mbar_wait(&sh.z_done[held], held_use & 1, abortp, g.status, ERR_WG_STORE))
          mbar_arrive(&sh.slot_empty[held]);
      }
    }
    __syncwarp();
  } else if (warp == 11) {
    // (fwd_next) the forward MMAs of a tile, issued as soon as the epilogue has put the
    // updated bf16 tile into its slot; they read that tile and the next step's input tile beside it
    if (lane == 0 && fwd_next) {
      const uint32_t idesc_z = idesc_bf16_f32(kBM, g.batch);
      uint32_t tile_ctr = tile_base, item_ctr = item_base;
      bool ok = true;
      for (int item = vblock; item < g.items && ok; item += vgrid, ++item_ctr) {
        int p, m0, nt0, nt;
        decode(item, p, m0, nt0, nt);
        for (int j = 0; j < nt; ++j, ++tile_ctr) {
          const int s = tile_ctr % g.slots;
          if (!mbar_wait(&sh.out_full[s], (tile_ctr / g.slots) & 1, abortp, g.status, ERR_WG_MMA)) {
            ok = false;
            break;
          }
          // the previous item's accumulator must have been read before this item's first
          // forward MMA overwrites it
          if (j == 0 && !mbar_wait(&sh.z_empty, (item_ctr & 1) ^ 1, abortp, g.status, ERR_WG_MMA)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t base = smem_u32(slot_base + (size_t)s * slot_bytes);
          const uint64_t adesc = smem_desc_k_sw64(base + w16_off);
          const uint64_t bdesc = smem_desc_k_sw64(base + xn_off);
#pragma unroll
          for (int k = 0; k < kBN / 16; ++k)
            umma_bf16(tmem_base + kZCol, adesc + 2 * k, bdesc + 2 * k, idesc_z,
                      (uint32_t)((j | k) != 0));
          umma_commit(&sh.z_done[s]);
          if (j == nt - 1) umma_commit(&sh.z_full);
        }
      }
    }
    __syncwarp();
  } else if (fwd_next) {
    // warps 12-15: the forward accumulator of every work item.  One weight row per lane (warp w
    // reads TMEM lanes 32 (w % 4) ...), 32 batch columns at a time.
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const size_t tile_floats = (size_t)g.batch * kBM;
    uint32_t item_ctr = item_base;
    uint32_t split_ctr = 0;          // items so far that went through z_part / z_flag
    for (int item = vblock; item < g.items; item += vgrid, ++item_ctr) {
      int p, m0, nt0, nt;
      decode(item, p, m0, nt0, nt);
      const bool single = nt == g.n_tiles;     // the accumulator is the whole product
      const int mt = m0 / kBM;
      const int m = m0 + r;
      const bool row_ok = m < g.out_rows;
      const float bias = row_ok ? g.bias_rep[(size_t)p * g.rep_stride + g.bias_off + m] : 0.f;
      // A_l of the next step from 32 (or the last 16) finished columns of this lane's row
      auto emit = [&](int c0, const float* z) {
        if (!row_ok) return;
        const int nc = min(32, g.batch - c0);
        uint32_t h[16];
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) {
          const float a0 = z[2 * jj] + bias, a1 = z[2 * jj + 1] + bias;
          __nv_bfloat162 h2 = __floats2bfloat162_rn(a0 > 0.f ? a0 : 0.f, a1 > 0.f ? a1 : 0.f);
          h[jj] = *reinterpret_cast<uint32_t*>(&h2);
        }
        uint4* dmb = reinterpret_cast<uint4*>(g.out_mb + ((size_t)p * g.out_rows + m) * g.batch + c0);
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (8 * v < nc) dmb[v] = make_uint4(h[4 * v], h[4 * v + 1], h[4 * v + 2], h[4 * v + 3]);
        const __nv_bfloat16* hh = reinterpret_cast<const __nv_bfloat16*>(h);
        __nv_bfloat16* dbm = g.out_bm + ((size_t)p * g.batch + c0) * g.out_rows + m;
#pragma unroll
        for (int jj = 0; jj < 32; ++jj)
          if (jj < nc) dbm[(size_t)jj * g.out_rows] = hh[jj];
      };
      if (!mbar_wait_relaxed(&sh.z_full, item_ctr & 1, abortp, g.status, ERR_WG_EPILOGUE, 400)) break;
      tc_fence_after_sync();
      float* zbase = g.zpart + ((size_t)p * g.m_tiles + mt) * g.n_chunks * tile_floats + r;
      float* zp = zbase + (size_t)(nt0 / g.chunk) * tile_floats;
      for (int c0 = 0; c0 < g.batch; c0 += 32) {
        uint32_t acc[32];
        if (c0 + 32 <= g.batch) {
          tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + kZCol + (uint32_t)c0, acc);
        } else {                             // the batch is a multiple of 16
          uint32_t h16[16];
          tmem_ld_16cols(tmem_base + ((uint32_t)(q * 32) << 16) + kZCol + (uint32_t)c0, h16);
#pragma unroll
          for (int jj = 0; jj < 16; ++jj) { acc[jj] = h16[jj]; acc[16 + jj] = 0u; }
        }
        tmem_ld_wait();
        if (single) {
          emit(c0, reinterpret_cast<const float*>(acc));
        } else {
#pragma unroll
          for (int jj = 0; jj < 32; ++jj)
            if (c0 + jj < g.batch) zp[(size_t)(c0 + jj) * kBM] = __uint_as_float(acc[jj]);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.z_empty);
      if (single) continue;
      // Whichever item of the row tile gets here last finishes the row tile.  The 128 lanes'
      // partial-sum stores are ordered before one lane's gpu-scope release on the counter by the
      // block-scope arrive/wait on z_part (the orders compose); on the other side that lane's
      // acquire on the counter is ordered before the 128 lanes' loads by z_flag, and the loads
      // go to the L2 (no stale L1 line can serve them).
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.z_part);
      if (warp == 12 && lane == 0 &&
          mbar_wait(&sh.z_part, split_ctr & 1, abortp, g.status, ERR_WG_EPILOGUE)) {
        int* cnt = g.zcount + (size_t)p * g.m_tiles + mt;
        int old;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(cnt) : "memory");
        const int last = old == g.n_chunks - 1;
        if (last) *cnt = 0;
        sh.z_last = last;
        mbar_arrive(&sh.z_flag);
      }
      __syncwarp();
      if (!mbar_wait(&sh.z_flag, split_ctr & 1, abortp, g.status, ERR_WG_EPILOGUE)) break;
      ++split_ctr;
      if (!sh.z_last) continue;
      for (int c0 = 0; c0 < g.batch; c0 += 32) {
        float z[32];
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) z[jj] = 0.f;
        // two runs' loads in flight at a time; the sums are formed in ascending run order
        for (int nc = 0; nc < g.n_chunks; nc += 2) {
          const float* s0 = zbase + (size_t)nc * tile_floats + (size_t)c0 * kBM;
          const bool two = nc + 1 < g.n_chunks;
          float a[32], b[32];
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            const bool in = c0 + jj < g.batch;
            a[jj] = in ? __ldcg(s0 + (size_t)jj * kBM) : 0.f;
            b[jj] = in && two ? __ldcg(s0 + tile_floats + (size_t)jj * kBM) : 0.f;
          }
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            z[jj] += a[jj];
            if (two) z[jj] += b[jj];
          }
        }
        emit(c0, z);
      }
    }
  }
}

}  // namespace wgrad
}  // namespace mavg
