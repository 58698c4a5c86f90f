// Declarations shared by the files of the MLP learner level (batch.cu, mlp.cu, mlp_simt.cu,
// mlp_tc.cu).
#pragma once
#include "common.cuh"

namespace mavg {

// idx = lo_j + floor(u * len_j / 2^32), u = top 32 bits of the stream value (see mavg.h).
__device__ __forceinline__ int32_t sample_index(uint64_t seed, int64_t round, int j, int step,
                                                int s, int P, int64_t S) {
  int64_t lo = (int64_t)(((unsigned __int128)j * (unsigned __int128)S) / (unsigned)P);
  int64_t hi = (int64_t)(((unsigned __int128)(j + 1) * (unsigned __int128)S) / (unsigned)P);
  uint64_t key = fold(learner_key(seed, kTagBatch, (uint64_t)round, (uint64_t)j), (uint64_t)step);
  uint64_t u = fold(key, (uint64_t)s) >> 32;
  return (int32_t)(lo + (int64_t)((u * (uint64_t)(hi - lo)) >> 32));
}

// batch.cu
cudaError_t launch_batch_indices(mavg_ctx* c, int64_t round, int step, int j_first, int j_count,
                                 int32_t* idx, int32_t* labels);
cudaError_t launch_gather(mavg_ctx* c, const int32_t* idx, int quant, float* out_f32,
                          __nv_bfloat16* out_bf, __nv_bfloat16* out_bft);
cudaError_t launch_sample_gather(mavg_ctx* c, int64_t round, int step, int32_t* idx,
                                 int32_t* labels, __nv_bfloat16* out_bf, __nv_bfloat16* out_bft);
cudaError_t launch_softmax_ce(mavg_ctx* c, const float* logits, int ldz, const int32_t* labels,
                              float* loss_out, int loss_stride, float* dz_f32, int ld32,
                              __nv_bfloat16* dz_bf, int ldbf, __nv_bfloat16* dz_bft, int ldbft,
                              bool update_bias, const MomArgs& mom = MomArgs());

// CUDA-core path (mlp_simt.cu): fp32 arithmetic, or bf16-rounded operands with fp32 FMAs.
size_t simt_workspace_bytes(const mavg_config* cfg, size_t base, size_t* act_off);
cudaError_t simt_step(mavg_ctx* c, int64_t round, int step);

// Tensor-core path (mlp_tc.cu): tcgen05 GEMMs fed by TMA.
bool tc_shapes_ok(const mavg_config* cfg, std::string* why);
size_t tc_workspace_bytes(const mavg_config* cfg, size_t base, size_t* act_off);
mavg_status tc_setup(mavg_ctx* c);
void tc_teardown(mavg_ctx* c);
cudaError_t tc_refresh_shared_operands(mavg_ctx* c);
cudaError_t tc_step(mavg_ctx* c, int64_t round, int step);

// Fused last layer on CUDA cores (tail_fused.cu): forward, loss, dZ_L, dgrad through the layer
// and the bias steps of the last two layers, for the tensor-core path's bf16 operands.
struct TailLaunch {
  const __nv_bfloat16* a_bm;     // A_{L-1} [P, B, in]
  const __nv_bfloat16* w16;      // bf16 W_L of learner 0
  int64_t w16_stride;            // elements between learners' copies (0: shared copy)
  bool shared_w;                 // biases are read from w~ (first step of a round)
  const int32_t* labels;
  float* loss_out;
  int loss_stride;
  __nv_bfloat16* dz_t;           // out: dZ_L^T [P, C, B]
  __nv_bfloat16* dzp_bm;         // out: dZ_{L-1} [P, B, in] and its transpose [P, in, B]
  __nv_bfloat16* dzp_mb;
  float* part;                   // scratch of tail_fused_part_bytes()
  MomArgs mom;
};
bool tail_fused_supported(const mavg_config* cfg);
size_t tail_fused_part_bytes(const mavg_config* cfg);
cudaError_t tail_fused_prepare();
cudaError_t launch_tail_fused(mavg_ctx* c, const TailLaunch& t);    // the products, dZ, partial sums
cudaError_t launch_tail_finish(mavg_ctx* c, const TailLaunch& t);   // bias steps and loss from the partials

void tc_reset_counters(mavg_ctx* c);          // after an abandoned device-side wait
void tc_step_plan(mavg_ctx* c, int32_t* out);  // entries of mavg_plan_entry
int tc_get_w16_cur(mavg_ctx* c);            // which bf16 copy of the doubled layer is current
void tc_set_w16_cur(mavg_ctx* c, int cur);

inline bool use_tensor_cores(const mavg_config* cfg) { return cfg->gemm_bf16 == 1; }

}  // namespace mavg
