// MLP learner level: layout bookkeeping and the per-round loop over the K local steps of
// Algorithm 1, dispatching each step to the tensor-core or the CUDA-core kernels.
#include "mlp.cuh"

namespace mavg {

mavg_status mlp_validate(const mavg_config* cfg, std::string* why) {
  if (cfg->gemm_bf16 < 0 || cfg->gemm_bf16 > 2) {
    if (why) *why = "gemm_bf16 must be 0, 1 or 2";
    return MAVG_ERR_INVALID_ARG;
  }
  if ((int64_t)cfg->P * cfg->B >= ((int64_t)1 << 24)) {
    if (why) *why = "P*B is too large";
    return MAVG_ERR_UNSUPPORTED;
  }
  if (use_tensor_cores(cfg) && !tc_shapes_ok(cfg, why)) return MAVG_ERR_UNSUPPORTED;
  return MAVG_OK;
}

size_t mlp_workspace_bytes(const mavg_config* cfg, Workspace* ws, size_t base) {
  return use_tensor_cores(cfg) ? tc_workspace_bytes(cfg, base, &ws->act)
                               : simt_workspace_bytes(cfg, base, &ws->act);
}

mavg_status mlp_setup(mavg_ctx* c) {
  const mavg_config& cfg = c->cfg;
  c->layers.clear();
  int64_t off = 0;
  for (int l = 0; l < cfg.n_layers; ++l) {
    MlpLayer ly{};
    ly.in = cfg.dims[l];
    ly.out = cfg.dims[l + 1];
    ly.w_off = off;
    off += (int64_t)ly.in * ly.out;
    ly.b_off = off;
    off += ly.out;
    c->layers.push_back(ly);
  }
  if (use_tensor_cores(&cfg)) return tc_setup(c);
  return MAVG_OK;
}

void mlp_teardown(mavg_ctx* c) {
  if (c->mlp) tc_teardown(c);
}

cudaError_t mlp_refresh_shared_operands(mavg_ctx* c) {
  if (use_tensor_cores(&c->cfg)) return tc_refresh_shared_operands(c);
  return cudaSuccess;
}

cudaError_t mlp_local_steps(mavg_ctx* c, int64_t round) {
  for (int k = 1; k <= c->cfg.K; ++k) {
    cudaError_t e = use_tensor_cores(&c->cfg) ? tc_step(c, round, k) : simt_step(c, round, k);
    if (e != cudaSuccess) return e;
    c->replicas_equal_global = false;
  }
  return cudaSuccess;
}

cudaError_t mlp_indices_only(mavg_ctx* c, int64_t round, int learner, int step, int32_t* dev_out) {
  return launch_batch_indices(c, round, step, learner, 1, dev_out, nullptr);
}

}  // namespace mavg
