// Minibatch side of the learner level: "randomly sample a mini-batch of size B_n"
// (Algorithm 1) as a counter-based index stream, the gather of the sampled rows, and the softmax
// cross-entropy loss with its gradient (the 1/B_n mean of Algorithm 1's update).
#include <mutex>

#include "mlp.cuh"

namespace mavg {
namespace {

// One thread per (learner, slot).  Also fetches the label.
__global__ void k_batch_indices(int32_t* __restrict__ idx, int32_t* __restrict__ labels,
                                const int32_t* __restrict__ y, uint64_t seed, int64_t round,
                                const int64_t* __restrict__ round_ptr, int step, int P, int B,
                                int64_t S, int j_first, int j_count) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= j_count * B) return;
  if (round_ptr) round = *round_ptr;   // replayed launches read the round from device memory
  int j = j_first + t / B, s = t % B;
  int32_t i = sample_index(seed, round, j, step, s, P, S);
  idx[t] = i;
  if (labels) labels[t] = y[i];
}

template <typename TIN>
__device__ __forceinline__ float to_f32(TIN v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Row gather.  One block per sampled row.  Outputs (any may be null):
//   out_f32 [rows, d]  fp32 (rounded to bf16 values when quant)
//   out_bf  [rows, d]  bf16
//   out_bft [P, d, B]  bf16, the same rows transposed per learner
template <typename TIN>
__global__ void __launch_bounds__(256)
k_gather(const TIN* __restrict__ x, const int32_t* __restrict__ idx, int d, int B, int quant,
         float* __restrict__ out_f32, __nv_bfloat16* __restrict__ out_bf,
         __nv_bfloat16* __restrict__ out_bft) {
  const int row = blockIdx.x;
  const TIN* src = x + (size_t)idx[row] * d;
  const int p = row / B, s = row % B;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = to_f32<TIN>(src[i]);
    __nv_bfloat16 b = __float2bfloat16_rn(v);
    if (out_f32) out_f32[(size_t)row * d + i] = quant ? __bfloat162float(b) : v;
    if (out_bf) out_bf[(size_t)row * d + i] = b;
    if (out_bft) out_bft[((size_t)p * d + i) * B + s] = b;
  }
}

// Index stream and gather in one kernel, for bf16 operands: block (32, 8) handles 32 batch slots of
// learner blockIdx.z and 64 input columns; it writes the rows [P, B, d] and, through a
// shared-memory tile, their transpose [P, d, B].  Blocks of the first column chunk also write the
// indices and labels.  d is a multiple of 8, B a multiple of 16.
template <typename TIN>
__global__ void __launch_bounds__(256)
k_sample_gather(const TIN* __restrict__ x, const int32_t* __restrict__ y, uint64_t seed,
                int64_t round, const int64_t* __restrict__ round_ptr, int step, int P, int B,
                int64_t S, int d, int32_t* __restrict__ idx_out, int32_t* __restrict__ labels_out,
                __nv_bfloat16* __restrict__ out_bf, __nv_bfloat16* __restrict__ out_bft) {
  __shared__ int32_t sidx[32];
  __shared__ __nv_bfloat16 tile[32][66];
  const int p = blockIdx.z, s0 = blockIdx.x * 32, c0 = blockIdx.y * 64;
  const int tx = threadIdx.x, ty = threadIdx.y;
  if (round_ptr) round = *round_ptr;
  if (ty == 0) {
    const int s = s0 + tx;
    int32_t i = 0;
    if (s < B) {
      i = sample_index(seed, round, p, step, s, P, S);
      if (blockIdx.y == 0) {
        idx_out[p * B + s] = i;
        labels_out[p * B + s] = y[i];
      }
    }
    sidx[tx] = i;
  }
  __syncthreads();
  const int c = c0 + 2 * tx;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int sl = ty + 8 * r, s = s0 + sl;
    __nv_bfloat16 v0 = __float2bfloat16_rn(0.f), v1 = v0;
    if (s < B && c < d) {                      // d is even: c + 1 < d as well
      const TIN* src = x + (size_t)sidx[sl] * d + c;
      v0 = __float2bfloat16_rn(to_f32<TIN>(src[0]));
      v1 = __float2bfloat16_rn(to_f32<TIN>(src[1]));
      __nv_bfloat162 pr;
      pr.x = v0; pr.y = v1;
      *reinterpret_cast<__nv_bfloat162*>(out_bf + ((size_t)p * B + s) * d + c) = pr;
    }
    tile[sl][2 * tx] = v0;
    tile[sl][2 * tx + 1] = v1;
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int cl = ty + 8 * r, cc = c0 + cl, s = s0 + tx;
    if (cc < d && s < B) out_bft[((size_t)p * d + cc) * B + s] = tile[tx][cl];
  }
}

// Softmax cross-entropy of learner blockIdx.x's B rows.  logits [P*B, ldz] fp32.
//   loss_out[p*loss_stride] = (1/B) sum_b (logsumexp(z_b) - z_b[y_b])
//   dz_f32 [P*B, ld32]  (softmax - onehot)/B
//   dz_bf  [P*B, ldbf], dz_bft [P, C rows of ldbft] bf16 copies   (may be null)
//   rep    if not null, the last layer's bias of learner p takes its SGD step here:
//          b[c] -= gamma * sum_b dz[b,c]  (ascending b, from the unrounded dz)
__global__ void __launch_bounds__(256)
k_softmax_ce(const float* __restrict__ logits, int ldz, const int32_t* __restrict__ labels, int B,
             int C, float* __restrict__ loss_out, int loss_stride, float* __restrict__ dz_f32,
             int ld32, __nv_bfloat16* __restrict__ dz_bf, int ldbf,
             __nv_bfloat16* __restrict__ dz_bft, int ldbft, float* __restrict__ rep,
             int64_t rep_stride, int64_t bias_off, float gamma, const MomArgs mom) {
  extern __shared__ float part[];     // [blockDim.x] loss partials
  const int p = blockIdx.x;
  const float inv_b = 1.0f / (float)B;
  float my_loss = 0.f;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    const size_t row = (size_t)p * B + b;
    const float* z = logits + row * ldz;
    float m = z[0];
    for (int c = 1; c < C; ++c) m = fmaxf(m, z[c]);
    float se = 0.f;
    for (int c = 0; c < C; ++c) se += expf(z[c] - m);
    const float lse = m + logf(se);
    const int yb = labels[row];
    my_loss += lse - z[yb];
    for (int c = 0; c < C; ++c) {
      float g = (expf(z[c] - lse) - (c == yb ? 1.f : 0.f)) * inv_b;
      dz_f32[row * ld32 + c] = g;
      __nv_bfloat16 gq = __float2bfloat16_rn(g);
      if (dz_bf) dz_bf[row * ldbf + c] = gq;
      if (dz_bft) dz_bft[((size_t)p * C + c) * ldbft + b] = gq;
    }
  }
  part[threadIdx.x] = my_loss;
  __syncthreads();   // also makes this block's dz_f32 stores visible to its own threads
  // fixed-order sums by one thread per output: B and C are small
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int t = 0; t < (int)blockDim.x; ++t) s += part[t];
    loss_out[(size_t)p * loss_stride] = s * inv_b;
  }
  if (rep) {
    float* bias = rep + (size_t)p * rep_stride + bias_off;
    float* ub = mom.u ? mom.u + (size_t)p * mom.u_stride + bias_off : nullptr;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
      float s = 0.f;
      for (int b = 0; b < B; ++b) s += dz_f32[((size_t)p * B + b) * ld32 + c];
      local_update(bias + c, bias[c], ub ? ub + c : nullptr, mom.read_u, s, gamma, mom.beta);
    }
  }
}

}  // namespace

cudaError_t launch_batch_indices(mavg_ctx* c, int64_t round, int step, int j_first, int j_count,
                                 int32_t* idx, int32_t* labels) {
  const int total = j_count * c->cfg.B;
  prof_begin(c, MAVG_K_BATCH);
  k_batch_indices<<<(total + 255) / 256, 256, 0, c->stream>>>(
      idx, labels, c->cfg.y, c->cfg.seed, round,
      c->capturing ? (const int64_t*)(ws_ptr(c, c->ws.status) + 64) : nullptr, step, c->cfg.P,
      c->cfg.B, c->cfg.n_samples, j_first, j_count);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_sample_gather(mavg_ctx* c, int64_t round, int step, int32_t* idx,
                                 int32_t* labels, __nv_bfloat16* out_bf, __nv_bfloat16* out_bft) {
  const int P = c->cfg.P, B = c->cfg.B, d = c->cfg.dims[0];
  dim3 grid((B + 31) / 32, (d + 63) / 64, P), block(32, 8);
  const int64_t* rp = c->capturing ? (const int64_t*)(ws_ptr(c, c->ws.status) + 64) : nullptr;
  prof_begin(c, MAVG_K_BATCH);
  if (c->cfg.x_dtype == MAVG_X_BF16)
    k_sample_gather<__nv_bfloat16><<<grid, block, 0, c->stream>>>(
        (const __nv_bfloat16*)c->cfg.x, c->cfg.y, c->cfg.seed, round, rp, step, P, B,
        c->cfg.n_samples, d, idx, labels, out_bf, out_bft);
  else
    k_sample_gather<float><<<grid, block, 0, c->stream>>>(
        (const float*)c->cfg.x, c->cfg.y, c->cfg.seed, round, rp, step, P, B, c->cfg.n_samples, d,
        idx, labels, out_bf, out_bft);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_gather(mavg_ctx* c, const int32_t* idx, int quant, float* out_f32,
                          __nv_bfloat16* out_bf, __nv_bfloat16* out_bft) {
  const int rows = c->cfg.P * c->cfg.B, d = c->cfg.dims[0];
  prof_begin(c, MAVG_K_BATCH);
  if (c->cfg.x_dtype == MAVG_X_BF16)
    k_gather<__nv_bfloat16><<<rows, 256, 0, c->stream>>>((const __nv_bfloat16*)c->cfg.x, idx, d,
                                                         c->cfg.B, quant, out_f32, out_bf, out_bft);
  else
    k_gather<float><<<rows, 256, 0, c->stream>>>((const float*)c->cfg.x, idx, d, c->cfg.B, quant,
                                                 out_f32, out_bf, out_bft);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_softmax_ce(mavg_ctx* c, const float* logits, int ldz, const int32_t* labels,
                              float* loss_out, int loss_stride, float* dz_f32, int ld32,
                              __nv_bfloat16* dz_bf, int ldbf, __nv_bfloat16* dz_bft, int ldbft,
                              bool update_bias, const MomArgs& mom) {
  const int P = c->cfg.P, B = c->cfg.B, C = c->cfg.dims[c->cfg.n_layers];
  int threads = 32;
  while (threads < B && threads < 256) threads <<= 1;
  size_t smem = (size_t)threads * sizeof(float);
  const MlpLayer& last = c->layers.back();
  prof_begin(c, MAVG_K_LOSS);
  k_softmax_ce<<<P, threads, smem, c->stream>>>(
      logits, ldz, labels, B, C, loss_out, loss_stride, dz_f32, ld32, dz_bf, ldbf, dz_bft, ldbft,
      update_bias ? c->buf.replicas : nullptr, c->buf.replica_stride, last.b_off,
      c->cfg.local_lr, mom);
  prof_end(c);
  return cudaGetLastError();
}

}  // namespace mavg

namespace mavg {
// ------------------------------------------------------------------------------------------------
// mavg_batch_indices_noalloc: the index stream without a handle and without any allocation.
// The B indices are staged in a fixed array that lives in the library's device image (every GPU
// that loads the library carries these 256 KB until the process exits) and are then copied to
// the caller's host buffer.
namespace {

constexpr int kNoAllocMaxB = 65536;
static __device__ __align__(256) int32_t g_noalloc_idx[kNoAllocMaxB];

constexpr int kNoAllocMaxDevices = 64;
int32_t* g_noalloc_ptr[kNoAllocMaxDevices] = {};
std::mutex g_noalloc_mutex;

// In host code the array's name is only a handle for the runtime, not a device address; the
// address on the current device is looked up once per device and remembered.
cudaError_t noalloc_scratch(int device, int32_t** out) {
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[device]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_idx);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[device] = (int32_t*)ptr;
  }
  *out = g_noalloc_ptr[device];
  return cudaSuccess;
}

}  // namespace
}  // namespace mavg

extern "C" mavg_status mavg_batch_indices_noalloc(uint64_t seed, int64_t round, int32_t P,
                                                  int32_t learner, int32_t step,
                                                  int64_t n_samples, int32_t B, void* stream,
                                                  int32_t* out) {
  using namespace mavg;
  if (!out || round < 1 || step < 1 || P < 1 || learner < 0 || learner >= P || B < 1 ||
      n_samples < P || n_samples >= ((int64_t)1 << 31)) {
    set_thread_error("mavg_batch_indices_noalloc: bad round, P, learner, step, n_samples, B or out");
    return MAVG_ERR_INVALID_ARG;
  }
  if (B > kNoAllocMaxB) {
    set_thread_error("mavg_batch_indices_noalloc: B exceeds the built-in staging array of 65536 "
                     "indices; use mavg_get_batch_indices with a workspace instead");
    return MAVG_ERR_INVALID_ARG;
  }
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e == cudaSuccess && (device < 0 || device >= kNoAllocMaxDevices)) {
    set_thread_error("mavg_batch_indices_noalloc: device ordinal out of range");
    return MAVG_ERR_UNSUPPORTED;
  }
  int32_t* scratch = nullptr;
  if (e == cudaSuccess) e = noalloc_scratch(device, &scratch);
  cudaStream_t s = (cudaStream_t)stream;
  if (e == cudaSuccess) {
    k_batch_indices<<<(B + 255) / 256, 256, 0, s>>>(scratch, nullptr, nullptr, seed, round,
                                                    nullptr, step, P, B, n_samples, learner, 1);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(out, scratch, (size_t)B * sizeof(int32_t), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    set_thread_error(std::string("mavg_batch_indices_noalloc: ") + cudaGetErrorString(e));
    return MAVG_ERR_CUDA;
  }
  return MAVG_OK;
}
