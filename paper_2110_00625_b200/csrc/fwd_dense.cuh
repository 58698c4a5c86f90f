// Launch interface of the dense first-step forward product (fwd_dense.cu).
//
// At the first local step of a round every learner holds w~ (Algorithm 1: "set w^j = w~"), so a
// hidden layer's forward products of all P learners are ONE dense product
//   Z^T[out, P*B] = W~[out, in] . X[P*B, in]^T
// with the weights read once instead of once per learner.  It is the only place of the learner
// level where a weight byte meets more than B columns of batch.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mavg {

constexpr int kDenseCols = 256;   // batch rows (of all learners) per tile

struct DensePlan {
  bool ok;         // the launch pays: enough 128 x 256 tiles to occupy the GPU
  int m_tiles, n_tiles, nkb, stages;
  size_t smem;
};

DensePlan plan_fwd_dense(int out, int in, int B, int P, int sm_count);
cudaError_t fwd_dense_prepare();
// w: bf16 [1, out, in] copy of w~, box 64 x 128 (128B swizzle); x: bf16 [1, P*B, in] view of the
// layer's input of all learners, box 64 x 256 (128B swizzle).  bias: the layer's bias in w~.
// Writes relu(Z + b) as bf16 in both orientations: out_bm [P, B, out], out_mb [P, out, B].
cudaError_t launch_fwd_dense(mavg_ctx* c, const DensePlan& pl, const CUtensorMap& w,
                             const CUtensorMap& x, int out, const float* bias,
                             __nv_bfloat16* out_bm, __nv_bfloat16* out_mb);

}  // namespace mavg
