// C ABI of the M-AVG engine: argument checking, the workspace carve-up and the round scheduler
// (stream-ordered launches of the kernels in the other files).  See include/mavg.h for the
// contract of every entry point.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <set>
#include <new>

#include "common.cuh"
#include "tc_ptx.cuh"

using namespace mavg;

namespace {

thread_local std::string g_create_error;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

mavg_status fail(std::string* sink, mavg_status st, const std::string& msg) {
  if (sink) *sink = msg;
  return st;
}

// Everything that can be decided without touching a device.
mavg_status validate_config(const mavg_config* cfg, std::string* why) {
  if (!cfg) return fail(why, MAVG_ERR_INVALID_ARG, "config is NULL");
  if (cfg->P < 1 || cfg->P > 65535) return fail(why, MAVG_ERR_INVALID_ARG, "P must be in [1, 65535]");
  if (cfg->K < 1) return fail(why, MAVG_ERR_INVALID_ARG, "K must be >= 1");
  if (!std::isfinite(cfg->local_lr)) return fail(why, MAVG_ERR_INVALID_ARG, "local_lr is not finite");
  if (!std::isfinite(cfg->block_lr)) return fail(why, MAVG_ERR_INVALID_ARG, "block_lr is not finite");
  if (!(cfg->mu >= 0.f && cfg->mu < 1.f)) return fail(why, MAVG_ERR_INVALID_ARG, "mu must be in [0, 1)");
  if (cfg->n < 1) return fail(why, MAVG_ERR_INVALID_ARG, "n must be >= 1");
  if (cfg->defer_broadcast != 0 && cfg->defer_broadcast != 1)
    return fail(why, MAVG_ERR_INVALID_ARG, "defer_broadcast must be 0 or 1");
  if (!(cfg->learner_momentum >= 0.f && cfg->learner_momentum < 1.f))
    return fail(why, MAVG_ERR_INVALID_ARG, "learner_momentum must be in [0, 1)");
  if (cfg->learner_momentum_reset != 0 && cfg->learner_momentum_reset != 1)
    return fail(why, MAVG_ERR_INVALID_ARG, "learner_momentum_reset must be 0 or 1");
  if (cfg->l2_keep != 0 && cfg->l2_keep != 1)
    return fail(why, MAVG_ERR_INVALID_ARG, "l2_keep must be 0 or 1");
  if (cfg->learner_momentum != 0.f && cfg->objective == MAVG_OBJ_NONE)
    return fail(why, MAVG_ERR_INVALID_ARG, "learner_momentum needs a learner level (objective)");
  switch (cfg->objective) {
    case MAVG_OBJ_NONE:
      break;
    case MAVG_OBJ_PSEUDOGRAD:
      if (!std::isfinite(cfg->pseudo_grad_sigma) || cfg->pseudo_grad_sigma < 0.f)
        return fail(why, MAVG_ERR_INVALID_ARG, "pseudo_grad_sigma must be finite and >= 0");
      break;
    case MAVG_OBJ_MLP: {
      if (cfg->B < 1) return fail(why, MAVG_ERR_INVALID_ARG, "B must be >= 1");
      if (cfg->n_layers < 1 || cfg->n_layers > MAVG_MAX_LAYERS)
        return fail(why, MAVG_ERR_INVALID_ARG, "n_layers must be in [1, 8]");
      int64_t count = 0;
      for (int l = 0; l <= cfg->n_layers; ++l)
        if (cfg->dims[l] < 1) return fail(why, MAVG_ERR_INVALID_ARG, "every layer width must be >= 1");
      for (int l = 0; l < cfg->n_layers; ++l)
        count += (int64_t)cfg->dims[l + 1] * cfg->dims[l] + cfg->dims[l + 1];
      if (count != cfg->n)
        return fail(why, MAVG_ERR_INVALID_ARG, "n does not match the MLP layout's parameter count");
      if (cfg->n_samples < cfg->P || cfg->n_samples >= (int64_t)1 << 31)
        return fail(why, MAVG_ERR_INVALID_ARG, "n_samples must be in [P, 2^31)");
      if (!cfg->x || !cfg->y) return fail(why, MAVG_ERR_BAD_BUFFER, "x or y is NULL");
      if (cfg->x_dtype != MAVG_X_F32 && cfg->x_dtype != MAVG_X_BF16)
        return fail(why, MAVG_ERR_INVALID_ARG, "unknown x_dtype");
      if (cfg->x_dtype == MAVG_X_BF16 && !cfg->gemm_bf16)
        return fail(why, MAVG_ERR_INVALID_ARG, "bf16 inputs need gemm_bf16");
      if ((uintptr_t)cfg->x % 16 || (uintptr_t)cfg->y % 4)
        return fail(why, MAVG_ERR_BAD_BUFFER, "x must be 16-byte aligned and y 4-byte aligned");
      return mlp_validate(cfg, why);
    }
    default:
      return fail(why, MAVG_ERR_INVALID_ARG, "unknown objective");
  }
  return MAVG_OK;
}

void carve_workspace(const mavg_config* cfg, Workspace* ws) {
  size_t off = 0;
  ws->status = off;
  off = align_up(off + 64 * sizeof(int32_t), 256);
  ws->losses = off;
  off = align_up(off + (size_t)cfg->P * cfg->K * sizeof(float), 256);
  ws->loss_mean = off;
  off = align_up(off + 64, 256);
  if (cfg->objective == MAVG_OBJ_MLP) {
    ws->idx = off;
    off = align_up(off + (size_t)cfg->P * cfg->B * sizeof(int32_t), 256);
    ws->labels = off;
    off = align_up(off + (size_t)cfg->P * cfg->B * sizeof(int32_t), 256);
    off = mlp_workspace_bytes(cfg, ws, off);
  }
  ws->total = off;
}

mavg_status set_err(mavg_ctx* c, mavg_status st, const std::string& msg) {
  c->err = msg;
  return st;
}

mavg_status cuda_fail(mavg_ctx* c, cudaError_t e, const char* where) {
  c->sticky = MAVG_ERR_CUDA;
  c->err = std::string(where) + ": " + cudaGetErrorString(e);
  return MAVG_ERR_CUDA;
}

#define CHECK_HANDLE(h)                          \
  do {                                           \
    if (!(h)) return MAVG_ERR_INVALID_ARG;       \
    if ((h)->sticky != MAVG_OK) return (h)->sticky; \
  } while (0)

#define CU(c, call, where)                                   \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) return cuda_fail((c), e__, where); \
  } while (0)

// mean of the P*K per-step losses, on the device, into ws.loss_mean
__global__ void k_mean_loss(const float* __restrict__ losses, int count, float* __restrict__ out) {
  __shared__ float part[32];
  float acc = 0.f;
  for (int i = threadIdx.x; i < count; i += blockDim.x) acc += losses[i];
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float s = threadIdx.x < (blockDim.x >> 5) ? part[threadIdx.x] : 0.f;
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) out[0] = s / (float)count;
  }
}

// A wait that cannot be satisfied: one warp, a barrier that expects an arrival nobody makes.  The
// bounded wait gives up after the handle's limit, records `code` and the kernel returns.
__global__ void k_selftest_wait(int* status, int code) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) tc::mbar_wait(&bar, 0, &abort_flag, status, code);
  __syncwarp();
}

mavg_status do_local_steps(mavg_ctx* c) {
  if (c->cfg.objective == MAVG_OBJ_NONE)
    return set_err(c, MAVG_ERR_STATE, "this handle has no learner level (MAVG_OBJ_NONE)");
  const int64_t round = c->round + 1;
  if (c->cfg.objective == MAVG_OBJ_PSEUDOGRAD) {
    CU(c, launch_pseudograd_steps(c, round), "pseudo-gradient local steps");
  } else {
    CU(c, mlp_local_steps(c, round), "MLP local steps");
  }
  c->replicas_equal_global = false;
  c->replicas_materialized = true;
  return MAVG_OK;
}

mavg_status do_meta_update(mavg_ctx* c) {
  // a meta-update with no local step since the last one averages P copies of w~ (d = 0); with
  // deferred copies they have to be written first.  Without a learner level the caller wrote
  // the replicas.
  if (c->cfg.objective != MAVG_OBJ_NONE && c->replicas_equal_global && !c->replicas_materialized)
    CU(c, launch_broadcast(c, false, /*force_copies=*/true), "re-broadcast");
  CU(c, launch_meta_update(c), "meta-update");
  c->round += 1;
  c->replicas_equal_global = true;
  if (c->cfg.objective == MAVG_OBJ_MLP && !c->shadow_fresh)
    CU(c, mlp_refresh_shared_operands(c), "operand refresh after the meta-update");
  c->shadow_fresh = false;
  return MAVG_OK;
}

mavg_status read_mean_loss(mavg_ctx* c, float* mean_loss) {
  if (c->cfg.objective == MAVG_OBJ_MLP) {
    float* lm = (float*)ws_ptr(c, c->ws.loss_mean);
    prof_begin(c, MAVG_K_LOSS);
    k_mean_loss<<<1, 256, 0, c->stream>>>((const float*)ws_ptr(c, c->ws.losses),
                                          c->cfg.P * c->cfg.K, lm);
    prof_end(c);
    CU(c, cudaGetLastError(), "mean-loss kernel");
    CU(c, cudaMemcpyAsync(mean_loss, lm, sizeof(float), cudaMemcpyDeviceToHost, c->stream),
       "loss read-back");
    CU(c, cudaStreamSynchronize(c->stream), "stream synchronize");
  } else {
    CU(c, cudaStreamSynchronize(c->stream), "stream synchronize");
    *mean_loss = 0.f;
  }
  return MAVG_OK;
}

}  // namespace

namespace mavg {
void set_thread_error(const std::string& msg) { g_create_error = msg; }
}  // namespace mavg

namespace {

// The persisting-L2 limit belongs to the device's context, which every handle of the process on
// that device shares: it is raised to the largest request among the live handles and put back to
// what it was when the last of them goes.
struct KeepState {
  std::multiset<size_t> wants;
  size_t prev = 0;
};
std::mutex g_keep_mu;
std::map<int, KeepState> g_keep;

bool keep_apply(int dev, const KeepState& k) {
  int max_keep = 0;
  if (cudaDeviceGetAttribute(&max_keep, cudaDevAttrMaxPersistingL2CacheSize, dev) != cudaSuccess ||
      max_keep <= 0)
    return false;
  // never below what the context had before the first handle asked
  const size_t want = *k.wants.rbegin() > k.prev ? *k.wants.rbegin() : k.prev;
  return cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize,
                            want < (size_t)max_keep ? want : (size_t)max_keep) == cudaSuccess;
}

bool keep_acquire(int dev, size_t want) {
  std::lock_guard<std::mutex> lock(g_keep_mu);
  KeepState& k = g_keep[dev];
  if (k.wants.empty() && cudaDeviceGetLimit(&k.prev, cudaLimitPersistingL2CacheSize) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  k.wants.insert(want);
  if (keep_apply(dev, k)) return true;
  cudaGetLastError();
  k.wants.erase(k.wants.find(want));
  return false;
}

void keep_release(int dev, size_t want) {
  std::lock_guard<std::mutex> lock(g_keep_mu);
  KeepState& k = g_keep[dev];
  auto it = k.wants.find(want);
  if (it == k.wants.end()) return;
  k.wants.erase(it);
  if (k.wants.empty()) {
    cudaCtxResetPersistingL2Cache();
    cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, k.prev);
  } else {
    keep_apply(dev, k);
  }
  cudaGetLastError();
}

}  // namespace

extern "C" {

mavg_status mavg_workspace_bytes(const mavg_config* cfg, size_t* out_bytes) {
  if (!out_bytes) return fail(&g_create_error, MAVG_ERR_INVALID_ARG, "out_bytes is NULL");
  *out_bytes = 0;
  mavg_status st = validate_config(cfg, &g_create_error);
  if (st != MAVG_OK) return st;
  Workspace ws;
  carve_workspace(cfg, &ws);
  *out_bytes = ws.total;
  return MAVG_OK;
}

mavg_status mavg_create(const mavg_config* cfg, const mavg_buffers* buf, mavg_handle* out) {
  if (!out) return fail(&g_create_error, MAVG_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  mavg_status st = validate_config(cfg, &g_create_error);
  if (st != MAVG_OK) return st;
  if (!buf) return fail(&g_create_error, MAVG_ERR_INVALID_ARG, "buffers is NULL");
  if (!buf->replicas || !buf->global_w || !buf->momentum || !buf->workspace)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER, "a device buffer is NULL");
  if ((uintptr_t)buf->replicas % 16 || (uintptr_t)buf->global_w % 16 ||
      (uintptr_t)buf->momentum % 16 || (uintptr_t)buf->workspace % 256)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER,
                "replicas, global_w, momentum must be 16-byte aligned and workspace 256-byte aligned");
  if (buf->replica_stride < cfg->n || buf->replica_stride % 4)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER,
                "replica_stride must be >= n and a multiple of 4");
  if (cfg->learner_momentum != 0.f && !buf->learner_u)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER, "learner_momentum != 0 needs the learner_u buffer");
  if ((uintptr_t)buf->learner_u % 16)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER, "learner_u must be 16-byte aligned");
  Workspace ws;
  carve_workspace(cfg, &ws);
  if (buf->workspace_bytes < ws.total)
    return fail(&g_create_error, MAVG_ERR_BAD_BUFFER, "workspace is smaller than mavg_workspace_bytes");

  int dev = 0;
  cudaGetLastError();   // a stale non-sticky error of earlier, unrelated calls is not ours
  cudaError_t e = cudaGetDevice(&dev);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess)
    return fail(&g_create_error, MAVG_ERR_CUDA, std::string("no usable CUDA device: ") + cudaGetErrorString(e));
  if (prop.major != 10)
    return fail(&g_create_error, MAVG_ERR_UNSUPPORTED, "this library is built for sm_100a devices only");

  mavg_ctx* c = new (std::nothrow) mavg_ctx();
  if (!c) return fail(&g_create_error, MAVG_ERR_INVALID_ARG, "out of host memory");
  c->cfg = *cfg;
  c->buf = *buf;
  c->stream = (cudaStream_t)cfg->stream;
  c->ws = ws;
  c->sm_count = prop.multiProcessorCount;
  c->device = dev;
  c->l2_bytes = (size_t)prop.l2CacheSize;

  e = cudaMemsetAsync(ws_ptr(c, c->ws.status), 0, 256, c->stream);
  if (e == cudaSuccess)
    e = cudaMemsetAsync(ws_ptr(c, c->ws.losses), 0, (size_t)cfg->P * cfg->K * sizeof(float), c->stream);
  if (e == cudaSuccess && buf->learner_u && cfg->objective != MAVG_OBJ_NONE)
    e = cudaMemsetAsync(buf->learner_u, 0,
                        ((size_t)(cfg->P - 1) * buf->replica_stride + cfg->n) * sizeof(float), c->stream);
  if (e == cudaSuccess) e = launch_broadcast(c, /*zero_v=*/true);
  if (e != cudaSuccess) {
    g_create_error = std::string("initialisation: ") + cudaGetErrorString(e);
    delete c;
    return MAVG_ERR_CUDA;
  }
  if (cfg->objective == MAVG_OBJ_MLP) {
    st = mlp_setup(c);
    if (st == MAVG_OK && mlp_refresh_shared_operands(c) != cudaSuccess) {
      st = MAVG_ERR_CUDA;
      c->err = "operand refresh failed";
    }
    if (st != MAVG_OK) {
      g_create_error = c->err;
      mlp_teardown(c);
      delete c;
      return st;
    }
    if (c->cfg.l2_keep == 1 && c->cfg.gemm_bf16 == 1 && masters_fit_l2(c)) {   // opt-in, tensor-core path
      // Room in the L2 for the learners' masters (see mavg_create in mavg.h).  Without it the
      // keep hints of the weight-gradient kernels have no effect; a refusal only costs speed.
      const size_t want = (size_t)cfg->P * (size_t)buf->replica_stride * sizeof(float);
      if (keep_acquire(dev, want)) {
        c->l2_keep = true;
        c->l2_keep_want = want;
        c->device = dev;
      }
    }
  }
  *out = c;
  return MAVG_OK;
}

mavg_status mavg_local_steps(mavg_handle h) {
  CHECK_HANDLE(h);
  return do_local_steps(h);
}

mavg_status mavg_meta_update(mavg_handle h) {
  CHECK_HANDLE(h);
  return do_meta_update(h);
}

mavg_status mavg_materialize_replicas(mavg_handle h) {
  CHECK_HANDLE(h);
  if (h->replicas_equal_global && !h->replicas_materialized)
    CU(h, launch_broadcast(h, false, /*force_copies=*/true), "re-broadcast");
  return MAVG_OK;
}

mavg_status mavg_round(mavg_handle h, float* mean_loss) {
  CHECK_HANDLE(h);
  mavg_status st = do_local_steps(h);
  if (st != MAVG_OK) return st;
  st = do_meta_update(h);
  if (st != MAVG_OK) return st;
  if (mean_loss) return read_mean_loss(h, mean_loss);
  return MAVG_OK;
}

mavg_status mavg_round_host(mavg_handle h, float* w_host, float* v_host, float* mean_loss) {
  CHECK_HANDLE(h);
  if (!w_host || !v_host) return set_err(h, MAVG_ERR_INVALID_ARG, "w_host or v_host is NULL");
  if (h->cfg.objective == MAVG_OBJ_NONE)
    return set_err(h, MAVG_ERR_STATE, "this handle has no learner level (MAVG_OBJ_NONE)");
  const size_t bytes = (size_t)h->cfg.n * sizeof(float);
  if (!h->s_copy) {
    CU(h, cudaStreamCreateWithFlags(&h->s_copy, cudaStreamNonBlocking), "copy stream");
    CU(h, cudaEventCreateWithFlags(&h->ev_copy_fork, cudaEventDisableTiming), "copy event");
    CU(h, cudaEventCreateWithFlags(&h->ev_copy_done, cudaEventDisableTiming), "copy event");
  }
  // v is first needed by the meta-update: its upload follows whatever the caller's stream did with
  // the buffer before this call and runs beside the K local steps
  // (submitted after w~, which the copy engine then serves first)
  CU(h, cudaMemcpyAsync(h->buf.global_w, w_host, bytes, cudaMemcpyHostToDevice, h->stream), "w~ upload");
  CU(h, cudaEventRecord(h->ev_copy_fork, h->stream), "copy fork");
  CU(h, cudaStreamWaitEvent(h->s_copy, h->ev_copy_fork, 0), "copy fork");
  CU(h, cudaMemcpyAsync(h->buf.momentum, v_host, bytes, cudaMemcpyHostToDevice, h->s_copy), "v upload");
  CU(h, cudaEventRecord(h->ev_copy_done, h->s_copy), "copy join");
  CU(h, launch_broadcast(h, false), "re-broadcast");
  h->replicas_equal_global = true;
  if (h->cfg.objective == MAVG_OBJ_MLP)
    CU(h, mlp_refresh_shared_operands(h), "operand refresh");
  mavg_status st = do_local_steps(h);
  CU(h, cudaStreamWaitEvent(h->stream, h->ev_copy_done, 0), "copy join");   // also on an error return
  if (st != MAVG_OK) return st;
  st = do_meta_update(h);
  if (st != MAVG_OK) return st;
  CU(h, cudaMemcpyAsync(w_host, h->buf.global_w, bytes, cudaMemcpyDeviceToHost, h->stream), "w~ download");
  CU(h, cudaMemcpyAsync(v_host, h->buf.momentum, bytes, cudaMemcpyDeviceToHost, h->stream), "v download");
  float dummy = 0.f;
  st = read_mean_loss(h, mean_loss ? mean_loss : &dummy);
  return st;
}

mavg_status mavg_set_hparams(mavg_handle h, int32_t K, float local_lr, float block_lr, float mu) {
  CHECK_HANDLE(h);
  if (K < 1) return set_err(h, MAVG_ERR_INVALID_ARG, "K must be >= 1");
  if (K > h->cfg.K && h->cfg.objective == MAVG_OBJ_MLP) {
    // the loss buffer was sized for the K given at creation
    size_t need = (size_t)h->cfg.P * K * sizeof(float);
    if (h->ws.losses + need > h->ws.loss_mean)
      return set_err(h, MAVG_ERR_INVALID_ARG, "K may not exceed the K the workspace was sized for");
  }
  if (!std::isfinite(local_lr) || !std::isfinite(block_lr))
    return set_err(h, MAVG_ERR_INVALID_ARG, "learning rates must be finite");
  if (!(mu >= 0.f && mu < 1.f)) return set_err(h, MAVG_ERR_INVALID_ARG, "mu must be in [0, 1)");
  h->cfg.K = K;
  h->cfg.local_lr = local_lr;
  h->cfg.block_lr = block_lr;
  h->cfg.mu = mu;
  return MAVG_OK;
}

mavg_status mavg_set_learner_momentum(mavg_handle h, float beta, int32_t reset) {
  CHECK_HANDLE(h);
  if (!(beta >= 0.f && beta < 1.f))
    return set_err(h, MAVG_ERR_INVALID_ARG, "learner momentum must be in [0, 1)");
  if (reset != 0 && reset != 1) return set_err(h, MAVG_ERR_INVALID_ARG, "reset must be 0 or 1");
  if (beta != 0.f && (!h->buf.learner_u || h->cfg.objective == MAVG_OBJ_NONE))
    return set_err(h, MAVG_ERR_STATE, "this handle was created without the learner_u buffer");
  h->cfg.learner_momentum = beta;
  h->cfg.learner_momentum_reset = reset;
  return MAVG_OK;
}

mavg_status mavg_get_batch_indices(mavg_handle h, int64_t round, int32_t learner, int32_t step,
                                   int32_t* out) {
  CHECK_HANDLE(h);
  if (h->cfg.objective != MAVG_OBJ_MLP)
    return set_err(h, MAVG_ERR_STATE, "batch indices exist for the MLP objective only");
  if (!out || round < 1 || learner < 0 || learner >= h->cfg.P || step < 1)
    return set_err(h, MAVG_ERR_INVALID_ARG, "bad round, learner, step or out");
  int32_t* dev = (int32_t*)ws_ptr(h, h->ws.idx);
  CU(h, mlp_indices_only(h, round, learner, step, dev), "index kernel");
  CU(h, cudaMemcpyAsync(out, dev, (size_t)h->cfg.B * sizeof(int32_t), cudaMemcpyDeviceToHost, h->stream),
     "index read-back");
  CU(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  return MAVG_OK;
}

mavg_status mavg_get_losses(mavg_handle h, float* out) {
  CHECK_HANDLE(h);
  if (!out) return set_err(h, MAVG_ERR_INVALID_ARG, "out is NULL");
  // only the MLP objective has a loss; for the others K may have grown past the K the loss
  // buffer was sized for (mavg_set_hparams bounds K for MLP handles only)
  if (h->cfg.objective != MAVG_OBJ_MLP)
    return set_err(h, MAVG_ERR_STATE, "minibatch losses exist for the MLP objective only");
  CU(h, cudaMemcpyAsync(out, ws_ptr(h, h->ws.losses), (size_t)h->cfg.P * h->cfg.K * sizeof(float),
                        cudaMemcpyDeviceToHost, h->stream), "loss read-back");
  CU(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  return MAVG_OK;
}

mavg_status mavg_get_round(mavg_handle h, int64_t* round) {
  CHECK_HANDLE(h);
  if (!round) return set_err(h, MAVG_ERR_INVALID_ARG, "round is NULL");
  *round = h->round;
  return MAVG_OK;
}

mavg_status mavg_set_round(mavg_handle h, int64_t round) {
  CHECK_HANDLE(h);
  if (round < 0) return set_err(h, MAVG_ERR_INVALID_ARG, "round must be >= 0");
  h->round = round;
  CU(h, launch_broadcast(h, false), "re-broadcast");
  h->replicas_equal_global = true;
  if (h->cfg.objective == MAVG_OBJ_MLP)
    CU(h, mlp_refresh_shared_operands(h), "operand refresh");
  return MAVG_OK;
}

mavg_status mavg_get_launch_count(mavg_handle h, int64_t* count) {
  if (!h || !count) return MAVG_ERR_INVALID_ARG;
  *count = h->launches;
  return MAVG_OK;
}

mavg_status mavg_get_step_plan(mavg_handle h, int32_t* out) {
  if (!h || !out) return MAVG_ERR_INVALID_ARG;
  for (int i = 0; i < MAVG_PLAN_COUNT; ++i) out[i] = 0;
  if (h->cfg.objective == MAVG_OBJ_MLP) mlp_step_plan(h, out);
  return MAVG_OK;
}

mavg_status mavg_set_profiling(mavg_handle h, int32_t on) {
  CHECK_HANDLE(h);
  h->profiling = on != 0;
  h->ev_open = nullptr;
  return MAVG_OK;
}

mavg_status mavg_set_schedule(mavg_handle h, int32_t mode) {
  CHECK_HANDLE(h);
  if (mode != MAVG_SCHED_GRAPH && mode != MAVG_SCHED_GRAPH_TC)
    return set_err(h, MAVG_ERR_INVALID_ARG, "schedule must be MAVG_SCHED_GRAPH (0) or MAVG_SCHED_GRAPH_TC (2)");
  h->schedule = mode;
  return MAVG_OK;
}

mavg_status mavg_get_profile(mavg_handle h, float* ms, int64_t* launches, int32_t reset) {
  CHECK_HANDLE(h);
  if (!ms || !launches) return set_err(h, MAVG_ERR_INVALID_ARG, "ms or launches is NULL");
  CU(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  for (int k = 0; k < MAVG_K_COUNT; ++k) { ms[k] = 0.f; launches[k] = 0; }
  for (const auto& sp : h->spans) {
    float t = 0.f;
    CU(h, cudaEventElapsedTime(&t, sp.a, sp.b), "event elapsed time");
    if (sp.cls >= 0 && sp.cls < MAVG_K_COUNT) { ms[sp.cls] += t; launches[sp.cls] += 1; }
  }
  if (reset) { h->spans.clear(); h->ev_used = 0; }
  return MAVG_OK;
}

mavg_status mavg_sync(mavg_handle h) {
  CHECK_HANDLE(h);
  int32_t flag = 0;
  CU(h, cudaMemcpyAsync(&flag, ws_ptr(h, h->ws.status), sizeof(flag), cudaMemcpyDeviceToHost, h->stream),
     "status read-back");
  CU(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  if (flag != 0) {
    char msg[96];
    snprintf(msg, sizeof msg, "a device-side wait ran out (code %d)", flag);
    cudaMemsetAsync(ws_ptr(h, h->ws.status), 0, sizeof(int32_t), h->stream);
    if (h->cfg.objective == MAVG_OBJ_MLP) mlp_reset_counters(h);
    return set_err(h, MAVG_ERR_TIMEOUT, msg);
  }
  return MAVG_OK;
}

mavg_status mavg_set_wait_limit(mavg_handle h, int32_t microseconds) {
  CHECK_HANDLE(h);
  if (microseconds < 0) return set_err(h, MAVG_ERR_INVALID_ARG, "the wait limit must be >= 0 microseconds");
  h->wait_limit_us = microseconds;
  // status[1] of the handle's status area; the copy is taken from pageable memory before the call returns
  CU(h, cudaMemcpyAsync(ws_ptr(h, h->ws.status) + sizeof(int32_t), &h->wait_limit_us, sizeof(int32_t),
                        cudaMemcpyHostToDevice, h->stream), "wait limit upload");
  return MAVG_OK;
}

mavg_status mavg_selftest_wait(mavg_handle h) {
  CHECK_HANDLE(h);
  k_selftest_wait<<<1, 32, 0, h->stream>>>((int*)ws_ptr(h, h->ws.status), 99);
  h->launches++;
  CU(h, cudaGetLastError(), "self-test kernel");
  return MAVG_OK;
}

const char* mavg_last_error(mavg_handle h) {
  if (!h) return g_create_error.c_str();
  return h->err.c_str();
}

mavg_status mavg_cache_release(mavg_handle h) {
  CHECK_HANDLE(h);
  CU(h, cudaStreamSynchronize(h->stream), "stream synchronize");
  if (h->l2_keep) CU(h, cudaCtxResetPersistingL2Cache(), "L2 reset");
  return MAVG_OK;
}

mavg_status mavg_destroy(mavg_handle h) {
  if (!h) return MAVG_OK;
  if (h->l2_keep) {
    cudaStreamSynchronize(h->stream);
    keep_release(h->device, h->l2_keep_want);
  }
  for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
  if (h->ev_copy_fork) cudaEventDestroy(h->ev_copy_fork);
  if (h->ev_copy_done) cudaEventDestroy(h->ev_copy_done);
  if (h->s_copy) cudaStreamDestroy(h->s_copy);
  mlp_teardown(h);
  delete h;
  return MAVG_OK;
}

}  // extern "C"
