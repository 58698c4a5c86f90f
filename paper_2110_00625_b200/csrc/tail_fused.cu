// Last layer of the MLP learner step in one CUDA-core kernel: forward product, softmax
// cross-entropy loss, dZ_L, the data gradient through the layer (with the ReLU mask of the layer
// below) and the two bias steps that hang on them.  With at most 32 classes these products are a
// few hundred thousand multiply-adds per learner -- far too small for a tensor-core tile each to
// pay for its launch and its tail -- so one block takes 8 batch rows of one learner through the
// whole sequence with the operands in shared memory:
//   z[b, c]      = sum_k A[b, k] W[c, k] + bias[c]                  (bf16 operands, fp32 sums)
//   loss_b       = logsumexp(z_b) - z_b[y_b];   dZ[b, c] = (softmax(z_b)[c] - [c == y_b]) / B
//   dA[b, k]     = sum_c bf16(dZ[b, c]) W[c, k];   dZprev[b, k] = A[b, k] > 0 ? dA[b, k] : 0
// and writes bf16(dZ) transposed (the weight-gradient kernel's operand), bf16(dZprev) in both
// orientations, and per-block partial sums of the loss and of the two bias gradients (from the
// unrounded dZ values).  A second small kernel adds the partials in ascending block order and
// takes the bias steps of Algorithm 1's local update; it runs beside the rest of the backward
// pass, which needs dZ_{L-1} but neither the biases nor the loss.
#include "mlp.cuh"

namespace mavg {
namespace {

constexpr int kRows = 8;         // batch rows per block (a multiple of 8: 16-byte transposed stores)
constexpr int kThreads = 256;
constexpr int kMaxC = 32;
static_assert(kThreads == 32 * kRows && kMaxC <= 32, "one warp per batch row, one lane per class");

struct TailArgs {
  const __nv_bfloat16* a_bm;     // A_{L-1} [P, B, in]
  const __nv_bfloat16* w16;      // W_L as bf16 [C, in]: w16 + p * w16_stride
  int64_t w16_stride;            // 0: one copy shared by all learners
  const float* bias_in;          // biases are read at bias_in[p * bias_in_stride + offset + i]
  int64_t bias_in_stride;        //   (the masters, or w~ with stride 0 at a round's first step)
  float* rep;                    // masters [P, rep_stride]: where the stepped biases are written
  int64_t rep_stride;
  int64_t b_off, bprev_off;      // offsets of b_L and b_{L-1} inside a replica
  const int32_t* labels;         // [P*B]
  float* loss_out;               // loss_out[p * loss_stride]
  int loss_stride;
  __nv_bfloat16* dz_t;           // dZ_L transposed [P, C, B]
  __nv_bfloat16* dzp_bm;         // dZ_{L-1} [P, B, in]     (null for a one-layer model)
  __nv_bfloat16* dzp_mb;         // dZ_{L-1} transposed [P, in, B]
  float* part;                   // [P, blocks, in + C + 1] partial sums
  int B, in, C;
  float gamma;
  MomArgs mom;
};

__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

// grid (B / kRows, P), a warp per batch row.  Dynamic shared memory: W [C, in] bf16, A [kRows, in] bf16.
__global__ void __launch_bounds__(kThreads)
k_last_layer_fused(const TailArgs g) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __shared__ float z[kRows][kMaxC + 1];     // logits, then unrounded dZ
  __shared__ __align__(16) float zq[kMaxC][kRows];   // dZ rounded to bf16 values, class-major
  __shared__ float row_loss[kRows];
  __shared__ float bias_s[kMaxC];
  __shared__ int label_s[kRows];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int p = blockIdx.y, blk = blockIdx.x, nblk = gridDim.x;
  const int r0 = blk * kRows;
  const int in = g.in, C = g.C, B = g.B;
  __nv_bfloat16* Ws = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* As = Ws + (size_t)C * in;

  // operands into shared memory, 16 bytes per load (in is a multiple of 8); the layer's bias and
  // the rows' labels too, so that no later phase waits for a global load of its own
  const float* bias_in = g.bias_in + (size_t)p * g.bias_in_stride;
  if (tid < C) bias_s[tid] = bias_in[g.b_off + tid];
  if (tid >= 32 && tid < 32 + kRows) label_s[tid - 32] = g.labels[(size_t)p * B + r0 + tid - 32];
  {
    // W and the rows as one list of 16-byte pieces; a thread has up to six loads in flight before
    // it stores the first (written as a plain copy loop, each load would wait for the store before)
    const uint4* wsrc = reinterpret_cast<const uint4*>(g.w16 + (size_t)p * g.w16_stride);
    const uint4* asrc = reinterpret_cast<const uint4*>(g.a_bm + ((size_t)p * B + r0) * in);
    uint4* dst = reinterpret_cast<uint4*>(Ws);            // A follows W in shared memory
    const int nw = C * in / 8, total = nw + kRows * in / 8;
    for (int i0 = tid; i0 < total; i0 += 6 * kThreads) {
      uint4 v[6];
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        const int i = i0 + j * kThreads;
        if (i < total) v[j] = i < nw ? wsrc[i] : asrc[i - nw];
      }
#pragma unroll
      for (int j = 0; j < 6; ++j) {
        const int i = i0 + j * kThreads;
        if (i < total) dst[i] = v[j];
      }
    }
  }
  __syncthreads();

  // forward: warp w takes row w; lanes split the contraction, two elements at a time.  Four
  // classes per pass: four independent chains, each the same sum in the same order as one chain
  // at a time would give.
  {
    const int r = warp;
    const uint32_t* arow = reinterpret_cast<const uint32_t*>(As + (size_t)r * in);
    for (int c = 0; c < C; c += 4) {
      const int c1 = min(c + 1, C - 1), c2 = min(c + 2, C - 1), c3 = min(c + 3, C - 1);
      const uint32_t* wrow0 = reinterpret_cast<const uint32_t*>(Ws + (size_t)c * in);
      const uint32_t* wrow1 = reinterpret_cast<const uint32_t*>(Ws + (size_t)c1 * in);
      const uint32_t* wrow2 = reinterpret_cast<const uint32_t*>(Ws + (size_t)c2 * in);
      const uint32_t* wrow3 = reinterpret_cast<const uint32_t*>(Ws + (size_t)c3 * in);
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      for (int k2 = lane; k2 < in / 2; k2 += 32) {
        const uint32_t x = arow[k2], w0 = wrow0[k2], w1 = wrow1[k2], w2 = wrow2[k2], w3 = wrow3[k2];
        a0 = fmaf(bf_lo(x), bf_lo(w0), a0);
        a1 = fmaf(bf_lo(x), bf_lo(w1), a1);
        a2 = fmaf(bf_lo(x), bf_lo(w2), a2);
        a3 = fmaf(bf_lo(x), bf_lo(w3), a3);
        a0 = fmaf(bf_hi(x), bf_hi(w0), a0);
        a1 = fmaf(bf_hi(x), bf_hi(w1), a1);
        a2 = fmaf(bf_hi(x), bf_hi(w2), a2);
        a3 = fmaf(bf_hi(x), bf_hi(w3), a3);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        a0 += __shfl_xor_sync(0xffffffffu, a0, o);
        a1 += __shfl_xor_sync(0xffffffffu, a1, o);
        a2 += __shfl_xor_sync(0xffffffffu, a2, o);
        a3 += __shfl_xor_sync(0xffffffffu, a3, o);
      }
      if (lane == 0) {
        z[r][c] = a0 + bias_s[c];
        if (c + 1 < C) z[r][c + 1] = a1 + bias_s[c + 1];
        if (c + 2 < C) z[r][c + 2] = a2 + bias_s[c + 2];
        if (c + 3 < C) z[r][c + 3] = a3 + bias_s[c + 3];
      }
    }
  }
  __syncthreads();

  // softmax cross-entropy: warp r takes row r, lane l class l; maximum and sum of exponentials
  // by butterflies over the warp
  {
    const int r = warp, l = lane;
    const int yb = label_s[r];
    const bool h = l < C;
    const float v = h ? z[r][l] : -INFINITY;
    float mx = v;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = h ? __expf(v - mx) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const float lse = mx + __logf(se);
    if (h) {
      if (l == yb) row_loss[r] = lse - v;
      const float gr = (__expf(v - lse) - (l == yb ? 1.f : 0.f)) * (1.0f / (float)B);
      z[r][l] = gr;
      zq[l][r] = __bfloat162float(__float2bfloat16_rn(gr));
    }
  }
  __syncthreads();

  float* part = g.part + ((size_t)p * nblk + blk) * (in + C + 1);
  // dZ_L transposed: class c, this block's rows (contiguous, 16 bytes per 8 rows); partial bias gradient
  if (tid < C) {
    const int c = tid;
    uint32_t w[kRows / 2];
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kRows / 2; ++j) {
      __nv_bfloat162 h2 = __floats2bfloat162_rn(z[2 * j][c], z[2 * j + 1][c]);
      w[j] = *reinterpret_cast<uint32_t*>(&h2);
      s += z[2 * j][c];
      s += z[2 * j + 1][c];
    }
    uint4* dst = reinterpret_cast<uint4*>(g.dz_t + ((size_t)p * C + c) * B + r0);
#pragma unroll
    for (int v = 0; v < kRows / 8; ++v) dst[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
    part[in + c] = s;
  }
  if (tid == kThreads - 1) {
    float s = 0.f;
    for (int r = 0; r < kRows; ++r) s += row_loss[r];
    part[in + C] = s;
  }

  // data gradient through the layer, masked by the activation below; thread per input column
  if (g.dzp_bm) {
    for (int k = tid; k < in; k += kThreads) {
      float acc[kRows];
#pragma unroll
      for (int r = 0; r < kRows; ++r) acc[r] = 0.f;
      for (int c = 0; c < C; ++c) {
        const float wv = __bfloat162float(Ws[(size_t)c * in + k]);
        const float4* zc = reinterpret_cast<const float4*>(zq[c]);
#pragma unroll
        for (int r4 = 0; r4 < kRows / 4; ++r4) {
          const float4 q4 = zc[r4];
          acc[4 * r4 + 0] = fmaf(q4.x, wv, acc[4 * r4 + 0]);
          acc[4 * r4 + 1] = fmaf(q4.y, wv, acc[4 * r4 + 1]);
          acc[4 * r4 + 2] = fmaf(q4.z, wv, acc[4 * r4 + 2]);
          acc[4 * r4 + 3] = fmaf(q4.w, wv, acc[4 * r4 + 3]);
        }
      }
      float colsum = 0.f;
      uint32_t w[kRows / 2];
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const bool live = __bfloat162float(As[(size_t)r * in + k]) > 0.f;     // ReLU'(0) = 0
        acc[r] = live ? acc[r] : 0.f;
        colsum += acc[r];
        g.dzp_bm[((size_t)p * B + r0 + r) * in + k] = __float2bfloat16_rn(acc[r]);
      }
#pragma unroll
      for (int j = 0; j < kRows / 2; ++j) {
        __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[2 * j], acc[2 * j + 1]);
        w[j] = *reinterpret_cast<uint32_t*>(&h2);
      }
      uint4* dst = reinterpret_cast<uint4*>(g.dzp_mb + ((size_t)p * in + k) * B + r0);
#pragma unroll
      for (int v = 0; v < kRows / 8; ++v) dst[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
      part[k] = colsum;
    }
  }
}

// Second half, off the step's critical chain (nothing later in the step reads what it writes):
// block p adds the per-block partials of learner p in ascending block order and takes the bias
// steps of Algorithm 1's local update for the last two layers; it also writes the minibatch loss.
__global__ void __launch_bounds__(kThreads)
k_last_layer_finish(const TailArgs g, int nblk) {
  const int tid = threadIdx.x, p = blockIdx.x;
  const int in = g.in, C = g.C, B = g.B;
  const float* bias_in = g.bias_in + (size_t)p * g.bias_in_stride;
  const float* pp = g.part + (size_t)p * nblk * (in + C + 1);
  float* rep = g.rep + (size_t)p * g.rep_stride;
  float* urow = g.mom.u ? g.mom.u + (size_t)p * g.mom.u_stride : nullptr;
  const int n_sum = (g.dzp_bm ? in : 0);
  for (int i = tid; i < in + C + 1; i += kThreads) {
    if (i < in && i >= n_sum) continue;
    float s = 0.f;
#pragma unroll 4
    for (int b = 0; b < nblk; ++b) s += pp[(size_t)b * (in + C + 1) + i];
    if (i < in) {
      const int64_t o = g.bprev_off + i;
      local_update(rep + o, bias_in[o], urow ? urow + o : nullptr, g.mom.read_u, s, g.gamma, g.mom.beta);
    } else if (i < in + C) {
      const int64_t o = g.b_off + (i - in);
      local_update(rep + o, bias_in[o], urow ? urow + o : nullptr, g.mom.read_u, s, g.gamma, g.mom.beta);
    } else {
      g.loss_out[(size_t)p * g.loss_stride] = s / (float)B;
    }
  }
}

size_t tail_smem_bytes(int in, int C) { return ((size_t)C * in + (size_t)kRows * in) * 2; }

}  // namespace

bool tail_fused_supported(const mavg_config* cfg) {
  const int L = cfg->n_layers;
  const int in = cfg->dims[L - 1], C = cfg->dims[L];
  if (cfg->B % kRows != 0 || in % 8 != 0 || C > kMaxC) return false;
  return tail_smem_bytes(in, C) <= 160 * 1024;
}

size_t tail_fused_part_bytes(const mavg_config* cfg) {
  const int L = cfg->n_layers;
  return (size_t)cfg->P * (cfg->B / kRows) * (cfg->dims[L - 1] + cfg->dims[L] + 1) * sizeof(float);
}

cudaError_t tail_fused_prepare() {
  return cudaFuncSetAttribute(k_last_layer_fused, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              160 * 1024);
}

namespace {
TailArgs tail_args(mavg_ctx* c, const TailLaunch& t) {
  const mavg_config& cfg = c->cfg;
  const int L = cfg.n_layers;
  const MlpLayer& ly = c->layers[L - 1];
  TailArgs g{};
  g.a_bm = t.a_bm;
  g.w16 = t.w16;
  g.w16_stride = t.w16_stride;
  g.bias_in = t.shared_w ? c->buf.global_w : c->buf.replicas;
  g.bias_in_stride = t.shared_w ? 0 : c->buf.replica_stride;
  g.rep = c->buf.replicas;
  g.rep_stride = c->buf.replica_stride;
  g.b_off = ly.b_off;
  g.bprev_off = L >= 2 ? c->layers[L - 2].b_off : 0;
  g.labels = t.labels;
  g.loss_out = t.loss_out;
  g.loss_stride = t.loss_stride;
  g.dz_t = t.dz_t;
  g.dzp_bm = L >= 2 ? t.dzp_bm : nullptr;
  g.dzp_mb = L >= 2 ? t.dzp_mb : nullptr;
  g.part = t.part;
  g.B = cfg.B;
  g.in = ly.in;
  g.C = ly.out;
  g.gamma = cfg.local_lr;
  g.mom = t.mom;
  return g;
}
}  // namespace

cudaError_t launch_tail_fused(mavg_ctx* c, const TailLaunch& t) {
  const TailArgs g = tail_args(c, t);
  dim3 grid((unsigned)(c->cfg.B / kRows), (unsigned)c->cfg.P);
  prof_begin(c, MAVG_K_LOSS);
  k_last_layer_fused<<<grid, kThreads, tail_smem_bytes(g.in, g.C), c->stream>>>(g);
  prof_end(c);
  return cudaGetLastError();
}

cudaError_t launch_tail_finish(mavg_ctx* c, const TailLaunch& t) {
  const TailArgs g = tail_args(c, t);
  prof_begin(c, MAVG_K_LOSS);
  k_last_layer_finish<<<c->cfg.P, kThreads, 0, c->stream>>>(g, c->cfg.B / kRows);
  prof_end(c);
  return cudaGetLastError();
}

}  // namespace mavg
