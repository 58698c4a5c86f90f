// Launch interface of the streaming weight-gradient + SGD kernel (wgrad_tc.cu).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mavg {

struct WgradPlan {
  int nkb, m_tiles, n_tiles, chunk, n_chunks, items, slots, a_bufs, grid, w16_on_b;
  int whole_rows; // (learner, row tile) pairs taken as one run of all column tiles (plans made with
                  // fwd_next: whole waves of such items first, the remaining rows cut into runs)
  int xn_bytes;   // room in every slot for the next step's input tile (plans made with fwd_next)
  size_t smem;
};

constexpr int kWgradTileRows = 128;   // rows of out per tile (box rows of the dZ^T and master maps)
constexpr int kWgradTileCols = 32;    // columns of in per tile

// streaming: the learners' masters do not stay in the L2 from one step to the next, so the kernel
// is a stream through HBM; the ring is then kept shallow and the runs of column tiles short
// (measured on the large MLP, B = 64: 4 slots and runs of 4 to 8 tiles give 0.84 of the copy
// bandwidth against 0.80 with 6 slots and runs of 16, and 0.67 with 3 slots).
// fwd_next: the launch may also take the next step's forward product of this layer along (see
// launch_wgrad_stream): every slot gets room for a [B, 32] tile of the next step's input and the
// runs of column tiles get long.
WgradPlan plan_wgrad_stream(int out, int in, int B, int P, int sm_count, bool momentum = false,
                            bool streaming = false, bool fwd_next = false);
cudaError_t wgrad_stream_prepare();
// dzt: bf16 [P, out, B] box 64 x 128 (128B swizzle); at: bf16 [P, in, B] box 64 x 32 (128B swizzle);
// w32: fp32 [P, out, in] box 32 x 128 (128B swizzle); w16: bf16 [P, out, in] box 32 x 128
// (64B swizzle).  w32_shared, if given, is an fp32 [1, out, in] view of w~ with the same box: the
// masters are then loaded from it for every learner (first step of a round, all w^j = w~) and
// stored to w32 as always.  With learner-level momentum (mom.u set; the plan made with
// momentum = true) u32 is the fp32 [P, out, in] view of the buffers u^j with w32's box.
// fn (plans made with fwd_next only): the launch also forms the NEXT local step's forward product
// of this layer from the updated weight tiles while they are in shared memory,
//   Z^T[out, B] = W_new[out, in] . Xn[B, in]^T,       A_next = relu(Z + b)  (bf16),
// accumulated in tensor memory over each run of column tiles.  With several runs per row the
// runs leave fp32 partial sums in zpart and the run that finishes last adds them up in ascending
// run order (so the result does not depend on which one that was).
struct WgradFwdNext {
  const CUtensorMap* xn;   // bf16 [P, B, in]: the layer's input of the next step, box 32 x B (64B swizzle)
  float* zpart;            // P x row tiles x runs x B x 128 floats
  int* zcount;             // P x row tiles arrival counters, zero before (and again after) the launch
  int64_t bias_off;        // the layer's bias in a learner's master vector
  int out_rows;            // rows of the layer
  __nv_bfloat16* out_bm;   // A_next [P, B, out]
  __nv_bfloat16* out_mb;   // A_next [P, out, B]
  bool store_w16;          // false: the bf16 copy of the weights is not written (a layer whose
                           // copy nothing else reads before the next launch that writes it:
                           // layer 1, which has no dgrad product)
};
cudaError_t launch_wgrad_stream(mavg_ctx* c, const WgradPlan& w, const CUtensorMap& dzt,
                                const CUtensorMap& at, const CUtensorMap& w32,
                                const CUtensorMap& w16, const CUtensorMap* w32_shared = nullptr,
                                const CUtensorMap* u32 = nullptr, const MomArgs& mom = MomArgs(),
                                const WgradFwdNext* fn = nullptr);

// Several layers' weight-gradient + SGD tiles in one persistent launch (layers listed in the
// order their tiles should run).  All plans must come from the same batch size and momentum
// setting, which fixes the ring geometry.
struct WgradLayerRef {
  const WgradPlan* plan;
  const CUtensorMap *dzt, *at, *w32, *w16;
  const CUtensorMap* w32_shared;   // null: every learner loads its own masters
  const CUtensorMap* u32;          // learner momentum view (may be null without momentum)
};
// max_grid > 0 caps the number of blocks (a launch that shares the GPU with another kernel).
cudaError_t launch_wgrad_multi(mavg_ctx* c, int n, const WgradLayerRef* layers,
                               const MomArgs& mom = MomArgs(), int max_grid = 0);

}  // namespace mavg
