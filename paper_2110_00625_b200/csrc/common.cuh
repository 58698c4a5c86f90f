// Shared declarations of the M-AVG CUDA library: the context behind a handle, the workspace
// carve-up, the counter-based generator (device and host) and the launch entry points of each
// kernel file.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/mavg.h"

namespace mavg {

// ------------------------------------------------------------------ SplitMix64 as a counter RNG
// fold(s, c) = mix64(s + (c+1) G): the (c+1)-th SplitMix64 output from state s.
constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kTagBatch = 1, kTagPseudoGrad = 2;

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ uint64_t fold(uint64_t s, uint64_t c) {
  return mix64(s + (c + 1) * kGamma);
}
// key of the stream (tag, round n, learner j); one more fold with the step k completes it
__host__ __device__ __forceinline__ uint64_t learner_key(uint64_t seed, uint64_t tag, uint64_t n,
                                                         uint64_t j) {
  return fold(fold(fold(seed, tag), n), j);
}

// --------------------------------------------------------------------- learner-level update
// Algorithm 1's local step  w <- w - gamma g,  or with learner-level momentum (u != nullptr)
//   u <- beta u - gamma g;  w <- w + u
// on the buffers u^j, laid out like the replicas.  read_u == 0: the stored u counts as zero (the
// learners restart from w~ and the momentum is reset there), so it is written but not read.
struct MomArgs {
  float beta = 0.f;
  float* u = nullptr;
  int64_t u_stride = 0;
  int read_u = 0;
};
__device__ __forceinline__ void msgd(float& w, float& u, float grad, float gamma, float beta) {
  u = fmaf(-gamma, grad, beta * u);
  w += u;
}
// One scalar parameter at *wp (read from w_in), its momentum slot at *up (may be null).
__device__ __forceinline__ void local_update(float* wp, float w_in, float* up, int read_u,
                                             float grad, float gamma, float beta) {
  if (up) {
    float u = read_u ? *up : 0.f;
    msgd(w_in, u, grad, gamma, beta);
    *up = u;
    *wp = w_in;
  } else {
    *wp = fmaf(-gamma, grad, w_in);
  }
}

// ------------------------------------------------------------------------------------- context
struct MlpLayer {
  int in, out;
  int64_t w_off, b_off;      // offsets (floats) inside a replica
};

// bf16 copy of the global model's weight matrices (the tensor-core path's shared operand at the
// first step of a round): layer l's weights w[w_off[l] .. w_off[l] + total[l]) go to
// dst[sh_off[l] ..).  All offsets and lengths are multiples of 4 elements.
struct ShadowMap {
  __nv_bfloat16* dst = nullptr;
  int L = 0;
  int64_t w_off[MAVG_MAX_LAYERS] = {}, total[MAVG_MAX_LAYERS] = {}, sh_off[MAVG_MAX_LAYERS] = {};
};

struct Workspace {           // byte offsets into the caller's scratch buffer
  size_t status = 0;         // int32[64]: [0] code of the first wait that ran out; [1] wait limit in
                             // microseconds (0: default); bytes 64..71: round (int64)
  size_t losses = 0;         // float [P*K]
  size_t loss_mean = 0;      // float [1]
  size_t idx = 0;            // int32 [P*B] sample indices of the current step
  size_t labels = 0;         // int32 [P*B]
  size_t act = 0;            // activations and their gradients (see mlp files)
  size_t total = 0;
};

}  // namespace mavg

struct mavg_ctx {
  mavg_config cfg;
  mavg_buffers buf;
  cudaStream_t stream = nullptr;
  int64_t round = 0;          // completed meta-updates
  int64_t launches = 0;
  mavg_status sticky = MAVG_OK;
  std::string err;
  int sm_count = 148;
  int32_t wait_limit_us = 0;  // mirrored in status[1] on the device
  size_t l2_bytes = 0;
  bool replicas_equal_global = true;  // every learner's model is w~: true between a (re-)broadcast
                                      // and the next local step
  bool replicas_materialized = true;  // the replica array really holds those P copies (false at a
                                      // round boundary with defer_broadcast)
  mavg::Workspace ws;
  std::vector<mavg::MlpLayer> layers;
  void* mlp = nullptr;        // state of the MLP path (owned by mlp files)
  mavg::ShadowMap shadow;     // set by the tensor-core path; dst == nullptr otherwise
  bool shadow_fresh = false;  // the last meta-update wrote the bf16 copy of w~ itself
  // per-launch timing (mavg_set_profiling): one event pair per launch, summed per kernel class
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  struct Span { int cls; cudaEvent_t a, b; };
  std::vector<Span> spans;
  cudaEvent_t ev_open = nullptr;
  int cls_open = 0;
  // CUDA graph of one round's K local steps (MLP objective): captured once on a private stream,
  // replayed on the caller's stream; rebuilt when K or the local learning rate change
  int schedule = 0;           // MLP tensor-core path, see mavg_set_schedule
  bool capturing = false;
  bool graph_disabled = false;
  cudaGraphExec_t graph_exec = nullptr;
  cudaStream_t cap_stream = nullptr;
  int graph_K = 0;
  float graph_lr = 0.f;
  float graph_beta = 0.f;
  int graph_reset = 0;
  int graph_schedule = 0;
  int graph_w16_cur = 0;      // state of the doubled bf16 copy after the recorded steps
  int64_t graph_nodes = 0;
  // this handle holds a request on the context's persisting-L2 limit (given up by mavg_destroy)
  bool l2_keep = false;
  size_t l2_keep_want = 0;
  int device = 0;
  // mavg_round_host: the upload of v runs on a copy stream of its own, next to the local steps
  cudaStream_t s_copy = nullptr;
  cudaEvent_t ev_copy_fork = nullptr, ev_copy_done = nullptr;
};

namespace mavg {

// All learners' fp32 masters together fit in half the L2: a step's weight-gradient kernels then
// ask the L2 to keep them until the next step reads them again.
inline bool masters_fit_l2(const mavg_ctx* c) {
  return (size_t)c->cfg.P * (size_t)c->buf.replica_stride * sizeof(float) <= c->l2_bytes / 2;
}

// Momentum arguments of a local step; from_broadcast: the step starts from w^j = w~.
inline MomArgs mom_args(const mavg_ctx* c, bool from_broadcast) {
  MomArgs m;
  if (c->cfg.learner_momentum != 0.f) {
    m.beta = c->cfg.learner_momentum;
    m.u = c->buf.learner_u;
    m.u_stride = c->buf.replica_stride;
    m.read_u = (from_broadcast && c->cfg.learner_momentum_reset) ? 0 : 1;
  }
  return m;
}

// Every launcher enqueues on ctx->stream, adds to ctx->launches and returns the CUDA status of
// the launch (cudaGetLastError), nothing else.
// w^j <- w~ (or, with defer_broadcast, only the book-keeping for it) and optionally v <- 0
cudaError_t launch_broadcast(mavg_ctx* c, bool zero_v, bool force_copies = false);
cudaError_t launch_meta_update(mavg_ctx* c);
cudaError_t launch_pseudograd_steps(mavg_ctx* c, int64_t round);

// MLP path (mlp_*.cu)
mavg_status mlp_validate(const mavg_config* cfg, std::string* why);
size_t mlp_workspace_bytes(const mavg_config* cfg, Workspace* ws, size_t base);
mavg_status mlp_setup(mavg_ctx* c);
void mlp_teardown(mavg_ctx* c);
cudaError_t mlp_refresh_shared_operands(mavg_ctx* c);   // after w~ changed
cudaError_t mlp_local_steps(mavg_ctx* c, int64_t round);
void mlp_reset_counters(mavg_ctx* c);                    // after an abandoned device-side wait
void mlp_step_plan(mavg_ctx* c, int32_t* out);           // entries of mavg_plan_entry
cudaError_t mlp_indices_only(mavg_ctx* c, int64_t round, int learner, int step, int32_t* dev_out);

// Bracket every kernel launch: prof_begin before it, prof_end after it (counts the launch).
inline cudaEvent_t prof_event(mavg_ctx* c) {
  if (c->ev_used == c->ev_pool.size()) {
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    c->ev_pool.push_back(e);
  }
  return c->ev_pool[c->ev_used++];
}
inline void prof_begin(mavg_ctx* c, int cls) {
  if (!c->profiling) return;
  c->ev_open = prof_event(c);
  c->cls_open = cls;
  cudaEventRecord(c->ev_open, c->stream);
}
inline void prof_end(mavg_ctx* c) {
  c->launches++;
  if (!c->profiling || !c->ev_open) return;
  cudaEvent_t b = prof_event(c);
  cudaEventRecord(b, c->stream);
  c->spans.push_back({c->cls_open, c->ev_open, b});
  c->ev_open = nullptr;
}

// Message returned by mavg_last_error(NULL) on the calling thread.
void set_thread_error(const std::string& msg);

inline char* ws_ptr(mavg_ctx* c, size_t off) { return (char*)c->buf.workspace + off; }

}  // namespace mavg
