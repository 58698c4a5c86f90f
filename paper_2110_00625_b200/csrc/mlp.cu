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

void mlp_drop_graph(mavg_ctx* c);

void mlp_teardown(mavg_ctx* c) {
  mlp_drop_graph(c);
  if (c->mlp) tc_teardown(c);
}

void mlp_reset_counters(mavg_ctx* c) {
  if (c->mlp) tc_reset_counters(c);
}

void mlp_step_plan(mavg_ctx* c, int32_t* out) {
  if (c->mlp) tc_step_plan(c, out);
}

cudaError_t mlp_refresh_shared_operands(mavg_ctx* c) {
  if (use_tensor_cores(&c->cfg)) return tc_refresh_shared_operands(c);
  return cudaSuccess;
}

namespace {

__global__ void k_set_round(int64_t* dst, int64_t round) { *dst = round; }

cudaError_t run_steps(mavg_ctx* c, int64_t round) {
  for (int k = 1; k <= c->cfg.K; ++k) {
    cudaError_t e = use_tensor_cores(&c->cfg) ? tc_step(c, round, k) : simt_step(c, round, k);
    if (e != cudaSuccess) return e;
    c->replicas_equal_global = false;
  }
  return cudaSuccess;
}

void drop_graph(mavg_ctx* c) {
  if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
  c->graph_exec = nullptr;
}

// Records the K steps of a round that starts from the broadcast state into a graph.  The steps
// are issued on a private capturing stream; nothing runs until the graph is launched.
cudaError_t build_graph(mavg_ctx* c, int64_t round) {
  drop_graph(c);
  cudaError_t e = cudaSuccess;
  if (!c->cap_stream) {
    e = cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) return e;
  }
  e = cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) return e;
  cudaStream_t user = c->stream;
  const int64_t before = c->launches;
  c->stream = c->cap_stream;
  c->capturing = true;
  c->replicas_equal_global = true;
  cudaError_t run = run_steps(c, round);
  c->capturing = false;
  c->stream = user;
  c->graph_nodes = c->launches - before;
  c->launches = before;
  cudaGraph_t graph = nullptr;
  e = cudaStreamEndCapture(c->cap_stream, &graph);
  if (run != cudaSuccess || e != cudaSuccess) {
    if (graph) cudaGraphDestroy(graph);
    return run != cudaSuccess ? run : e;
  }
  e = cudaGraphInstantiate(&c->graph_exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) {
    c->graph_exec = nullptr;
    return e;
  }
  c->graph_K = c->cfg.K;
  c->graph_lr = c->cfg.local_lr;
  c->graph_beta = c->cfg.learner_momentum;
  c->graph_reset = c->cfg.learner_momentum_reset;
  c->graph_schedule = c->schedule;
  c->graph_w16_cur = use_tensor_cores(&c->cfg) ? tc_get_w16_cur(c) : 0;
  return cudaSuccess;
}

}  // namespace

void mlp_drop_graph(mavg_ctx* c) {
  drop_graph(c);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  c->cap_stream = nullptr;
}

cudaError_t mlp_local_steps(mavg_ctx* c, int64_t round) {
  // The usual round starts from the broadcast state and is replayed from a graph.  Rounds that
  // start elsewhere (local steps called twice in a row), profiled rounds and handles whose
  // capture failed once take the launch-by-launch path.
  // The CUDA-core path reads every learner's own copy from the first step on: a deferred
  // re-broadcast (Algorithm 1, "set w^j = w~") is carried out here, on the caller's stream and
  // outside the recorded graph, so that a replay never depends on whether the copies happened to
  // exist when the graph was recorded.
  if (!use_tensor_cores(&c->cfg) && c->replicas_equal_global && !c->replicas_materialized) {
    cudaError_t e = launch_broadcast(c, false, /*force_copies=*/true);
    if (e != cudaSuccess) return e;
  }
  const bool want_graph = !c->profiling && !c->graph_disabled && c->replicas_equal_global;
  if (!want_graph) return run_steps(c, round);
  if (!c->graph_exec || c->graph_K != c->cfg.K || c->graph_lr != c->cfg.local_lr ||
      c->graph_beta != c->cfg.learner_momentum || c->graph_reset != c->cfg.learner_momentum_reset ||
      c->graph_schedule != c->schedule) {
    cudaError_t e = build_graph(c, round);
    if (e != cudaSuccess) {
      cudaGetLastError();
      c->graph_disabled = true;
      c->replicas_equal_global = true;
      return run_steps(c, round);
    }
  }
  k_set_round<<<1, 1, 0, c->stream>>>((int64_t*)(ws_ptr(c, c->ws.status) + 64), round);
  c->launches++;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = cudaGraphLaunch(c->graph_exec, c->stream);
  if (e != cudaSuccess) return e;
  c->launches += c->graph_nodes;
  c->replicas_equal_global = false;
  if (use_tensor_cores(&c->cfg)) tc_set_w16_cur(c, c->graph_w16_cur);
  return cudaSuccess;
}

cudaError_t mlp_indices_only(mavg_ctx* c, int64_t round, int learner, int step, int32_t* dev_out) {
  return launch_batch_indices(c, round, step, learner, 1, dev_out, nullptr);
}

}  // namespace mavg
