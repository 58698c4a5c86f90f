// Tensor-core MLP learner step (placeholder until the tcgen05 kernels land).
#include "mlp.cuh"

namespace mavg {
bool tc_shapes_ok(const mavg_config*, std::string* why) {
  if (why) *why = "tensor-core path not built";
  return false;
}
size_t tc_workspace_bytes(const mavg_config*, size_t base, size_t* act_off) { *act_off = base; return base; }
mavg_status tc_setup(mavg_ctx*) { return MAVG_ERR_UNSUPPORTED; }
void tc_teardown(mavg_ctx*) {}
cudaError_t tc_refresh_shared_operands(mavg_ctx*) { return cudaSuccess; }
cudaError_t tc_step(mavg_ctx*, int64_t, int) { return cudaErrorNotSupported; }
}  // namespace mavg
