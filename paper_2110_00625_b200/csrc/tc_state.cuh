// Host-side state of the tensor-core MLP path: workspace layout, launch plans and tensor maps.
// Built and used by mlp_tc.cu.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "fwd_dense.cuh"
#include "wgrad_tc.cuh"

namespace mavg {

struct TcLayout {
  int L;
  int cpad;                                  // last layer's dZ row length (multiple of 8)
  int64_t n16;                               // elements per bf16 copy row
  int64_t sh_off[MAVG_MAX_LAYERS];
  size_t xg[2], xt[2];                       // gathered batch, two buffers used by alternate steps
  size_t act[MAVG_MAX_LAYERS + 1], act_t[MAVG_MAX_LAYERS + 1];
  // second set of activation buffers: odd steps use it where a step's weight-gradient launches
  // already produce the next step's activations (TcState::fuse_upto)
  size_t act_b[MAVG_MAX_LAYERS + 1], act_t_b[MAVG_MAX_LAYERS + 1];
  size_t dz[MAVG_MAX_LAYERS + 1], dz_t[MAVG_MAX_LAYERS + 1];
  size_t part, part_bytes;
  size_t counters, counters_bytes;
  size_t w16, w16g;
  size_t tail_part;                          // partial sums of the fused last-layer kernel
  size_t zcount, zcount_bytes;               // arrival counters of those partial sums
  size_t zpart, zpart_bytes;                 // partial sums of a forward product that rides along
                                             // with a weight-gradient launch (wgrad_tc.cuh); one
                                             // layer at a time
  size_t w16b;                               // second bf16 copy of layer L-1's weights [P, w16b_stride]
  int64_t w16b_stride;
  size_t end;
};


struct GemmPlan { int m_tiles, n_tiles, splits, kb_per_split, nkb, BN, stages, two_per_sm; uint32_t tmem_cols; };

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  TcLayout lay;
  EncodeTiledFn encode = nullptr;
  // per layer l = 1..L (index l)
  CUtensorMap w[MAVG_MAX_LAYERS + 1], wg[MAVG_MAX_LAYERS + 1];       // [out, in] copies
  CUtensorMap act_in[MAVG_MAX_LAYERS + 1];    // [B, d_{l-1}] input activations of layer l >= 2
  CUtensorMap act_in_t[MAVG_MAX_LAYERS + 1];  // [d_{l-1}, B]
  CUtensorMap x_in[2], x_in_t[2];             // layer 1's input: the two gather buffers
  CUtensorMap dz[MAVG_MAX_LAYERS + 1];        // [B, d_l]
  CUtensorMap dz_t[MAVG_MAX_LAYERS + 1];      // [d_l, B]
  CUtensorMap w_mn[MAVG_MAX_LAYERS + 1], wg_mn[MAVG_MAX_LAYERS + 1];  // [out, in] copies, 64 x 64 boxes
  CUtensorMap w32[MAVG_MAX_LAYERS + 1];       // fp32 masters [out, in]: wgrad loads and stores
  CUtensorMap w32g[MAVG_MAX_LAYERS + 1];      // the same view of w~ (one copy): first-step loads
  CUtensorMap w16_st[MAVG_MAX_LAYERS + 1];    // store view of the bf16 copy
  CUtensorMap u32[MAVG_MAX_LAYERS + 1];       // learner momentum buffers, the masters' view
  bool wgrad_mom = false;                     // the wgrad plans leave room for the u tile
  // hidden-layer forward with the contraction split over a thread-block cluster (fwd_ks[l].splits
  // > 1 where used): plan and the input maps whose box is the whole batch high
  GemmPlan fwd_ks[MAVG_MAX_LAYERS + 1];
  CUtensorMap act_in_ks[MAVG_MAX_LAYERS + 1], x_in_ks[2];
  // Layer L-1's bf16 weights exist twice (L >= 3): where its weight gradient runs beside the
  // dgrad product that still reads the old copy, it writes the other one.  w16_cur says which
  // copy holds the current weights; *_b are the views of copy 1.
  int dbl_layer = 0;
  int w16_cur = 0;
  CUtensorMap w_b, w_mn_b, w16_st_b;
  bool tail_ok = false;                       // the fused last-layer kernel covers the shape
  bool wgrad_merged = false;                  // all layers' weight gradients in one launch
  // Forward products of step k+1 formed inside step k's weight-gradient launches (see
  // wgrad_tc.cuh), for layers 1..fuse_upto (0: none; at most L-1).  Possible where those launches
  // stand alone.  Step k then runs, after its dgrad chain, for l = 1..fuse_upto: weight gradient +
  // SGD of layer l with the forward product of W_l(k+1) and A_{l-1}(k+1) riding along, which
  // leaves A_l(k+1) behind.  Steps alternate between two sets of
  // activation buffers (A_l(k) is still read by layer l+1's weight gradient when A_l(k+1) is
  // written); *_b are the views of the second set, a_next[l][i] the input of layer l in set i
  // (l = 1: gather buffer i) as the riding product reads it.  fwd_done: how many leading
  // layers of the step about to be issued already have their activations; gathered_step: the
  // step whose batch has already been gathered by the launch-by-launch form.
  int fuse_upto = 0;
  int fwd_done = 0;
  int gathered_step = 0;
  CUtensorMap act_in_b[MAVG_MAX_LAYERS + 1], act_in_t_b[MAVG_MAX_LAYERS + 1],
      act_in_ks_b[MAVG_MAX_LAYERS + 1];
  CUtensorMap a_next[MAVG_MAX_LAYERS + 1][2];
  WgradPlan wgrad_f[MAVG_MAX_LAYERS + 1];     // plans of the launches that take a forward along
  // First local step of a round (all learners hold w~): hidden layer l's forward as one dense
  // product over the batch rows of all learners (fwd_dense.cuh) where dense[l].ok; in2d[l][i]:
  // the layer's input in buffer set i (l = 1: gather buffer i) as one [P*B, d_{l-1}] array.
  DensePlan dense[MAVG_MAX_LAYERS + 1];
  CUtensorMap in2d[MAVG_MAX_LAYERS + 1][2];
  GemmPlan fwd[MAVG_MAX_LAYERS + 1], dgrad[MAVG_MAX_LAYERS + 1];
  WgradPlan wgrad[MAVG_MAX_LAYERS + 1];
  // side streams and events for the branches of a step that may overlap
  cudaStream_t s_wgrad = nullptr, s_gather = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_wgrad_done = nullptr, ev_gather_done = nullptr,
              ev_x_free[2] = {nullptr, nullptr};
};


int tc_get_w16_cur(mavg_ctx* c);
void tc_set_w16_cur(mavg_ctx* c, int cur);

}  // namespace mavg
