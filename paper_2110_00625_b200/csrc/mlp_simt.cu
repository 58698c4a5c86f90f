// CUDA-core MLP learner step, batched over the P learners (blockIdx.z).
//   forward   Z_l = act(A_{l-1}) W_l^T + b_l                      (A_0 = gathered minibatch)
//   backward  dZ_{l-1} = (dZ_l W_l) .* [Z_{l-1} > 0];  dW_l = dZ_l^T act(A_{l-1});  db_l = colsum dZ_l
//   SGD       W_l <- W_l - gamma dW_l, b_l <- b_l - gamma db_l    (Algorithm 1's local update)
// fp32 FMAs throughout.  With QUANT every matrix-product operand is first rounded to bf16
// (nearest-even), which makes this path compute the same thing as the tensor-core path; it is the
// path for true fp32 models and for layer widths the tensor-core path does not cover.
// Buffers hold pre-activations Z_l and dZ_l in fp32; ReLU and rounding are applied on load.
#include "mlp.cuh"

namespace mavg {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

__device__ __forceinline__ float qbf(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

enum LoadOp { LD_PLAIN = 0, LD_RELU = 1 };

template <bool QUANT, int OP>
__device__ __forceinline__ float load_op(float v) {
  if (OP == LD_RELU) v = v > 0.f ? v : 0.f;
  return QUANT ? qbf(v) : v;
}

struct GemmArgs {
  const float* A; int64_t a_batch; int64_t a_m, a_k;   // A(m,k) = A[p*a_batch + m*a_m + k*a_k]
  const float* B; int64_t b_batch; int64_t b_n, b_k;   // B(n,k) = B[p*b_batch + n*b_n + k*b_k]
  int M, N, K;
  // epilogue operands
  float* C; int64_t c_batch; int64_t c_m;               // C(m,n) = C[p*c_batch + m*c_m + n]
  const float* aux; int64_t aux_batch; int64_t aux_m;   // bias [n] (fwd) or mask source Z (dgrad)
  float gamma;
  MomArgs mom;          // EPI_WGRAD_SGD: learner momentum slots at mom.u[p*u_stride + (C's offset)]
  int64_t u_off;        // offset of C inside a replica (the same inside u^j)
};

enum Epi { EPI_FWD = 0, EPI_DGRAD = 1, EPI_WGRAD_SGD = 2 };

// C(m,n) = sum_k opA(A(m,k)) * opB(B(n,k)), 64x64 tile, 256 threads, 4x4 outputs per thread.
template <bool QUANT, int OPA, int OPB, bool A_KC, bool B_KC, int EPI>
__global__ void __launch_bounds__(256) k_simt_gemm(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int p = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const float* A = g.A + (size_t)p * g.a_batch;
  const float* B = g.B + (size_t)p * g.b_batch;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;   // tx over n, ty over m
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.K; k0 += BK) {
    // 64 x 16 elements per operand, 4 per thread; consecutive threads follow the unit stride
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int lin = tid + e * 256;
      int mm, kk;
      if (A_KC) { kk = lin % BK; mm = lin / BK; } else { mm = lin % BM; kk = lin / BM; }
      int gm = m0 + mm, gk = k0 + kk;
      float v = 0.f;
      if (gm < g.M && gk < g.K) v = load_op<QUANT, OPA>(A[(size_t)gm * g.a_m + (size_t)gk * g.a_k]);
      As[kk][mm] = v;
      int nn;
      if (B_KC) { kk = lin % BK; nn = lin / BK; } else { nn = lin % BN; kk = lin / BN; }
      int gn = n0 + nn;
      gk = k0 + kk;
      v = 0.f;
      if (gn < g.N && gk < g.K) v = load_op<QUANT, OPB>(B[(size_t)gn * g.b_n + (size_t)gk * g.b_k]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  float* C = g.C + (size_t)p * g.c_batch;
  float* U = (EPI == EPI_WGRAD_SGD && g.mom.u) ? g.mom.u + (size_t)p * g.mom.u_stride + g.u_off
                                               : nullptr;
  const float* aux = g.aux ? g.aux + (size_t)p * g.aux_batch : nullptr;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    int gm = m0 + ty * TM + i;
    if (gm >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int gn = n0 + tx * TN + j;
      if (gn >= g.N) continue;
      float v = acc[i][j];
      size_t ci = (size_t)gm * g.c_m + gn;
      if (EPI == EPI_FWD) {
        C[ci] = v + aux[gn];
      } else if (EPI == EPI_DGRAD) {
        C[ci] = aux[(size_t)gm * g.aux_m + gn] > 0.f ? v : 0.f;   // ReLU'(0) = 0
      } else {
        local_update(C + ci, C[ci], U ? U + ci : nullptr, g.mom.read_u, v, g.gamma, g.mom.beta);
      }
    }
  }
}

// b[o] -= gamma * sum_b dZ[b, o], ascending b.  grid (ceil(out/256), P)
__global__ void __launch_bounds__(256)
k_simt_bias_sgd(const float* __restrict__ dz, int64_t dz_batch, int B, int out,
                float* __restrict__ rep, int64_t rep_stride, int64_t b_off, float gamma,
                const MomArgs mom) {
  int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= out) return;
  const int p = blockIdx.y;
  const float* d = dz + (size_t)p * dz_batch;
  float s = 0.f;
  for (int b = 0; b < B; ++b) s += d[(size_t)b * out + o];
  float* bias = rep + (size_t)p * rep_stride + b_off;
  float* ub = mom.u ? mom.u + (size_t)p * mom.u_stride + b_off : nullptr;
  local_update(bias + o, bias[o], ub ? ub + o : nullptr, mom.read_u, s, gamma, mom.beta);
}

struct SimtBuffers {
  float* xg;                      // [P, B, d0]
  float* z[MAVG_MAX_LAYERS + 1];  // z[l]  [P, B, d_l], l = 1..L
  float* dz[MAVG_MAX_LAYERS + 1]; // dz[l] [P, B, d_l]
};

SimtBuffers carve(const mavg_config* cfg, char* base) {
  SimtBuffers sb{};
  const size_t rows = (size_t)cfg->P * cfg->B;
  size_t off = 0;
  auto take = [&](size_t floats) {
    float* p = (float*)(base + off);
    off += (floats * sizeof(float) + 255) / 256 * 256;
    return p;
  };
  sb.xg = take(rows * cfg->dims[0]);
  for (int l = 1; l <= cfg->n_layers; ++l) {
    sb.z[l] = take(rows * cfg->dims[l]);
    sb.dz[l] = take(rows * cfg->dims[l]);
  }
  return sb;
}

template <bool QUANT>
cudaError_t step_impl(mavg_ctx* c, int64_t round, int step) {
  const mavg_config& cfg = c->cfg;
  const int P = cfg.P, B = cfg.B, L = cfg.n_layers;
  SimtBuffers sb = carve(&cfg, ws_ptr(c, c->ws.act));
  int32_t* idx = (int32_t*)ws_ptr(c, c->ws.idx);
  int32_t* labels = (int32_t*)ws_ptr(c, c->ws.labels);
  float* losses = (float*)ws_ptr(c, c->ws.losses);
  cudaError_t e;
  if ((e = launch_batch_indices(c, round, step, 0, P, idx, labels)) != cudaSuccess) return e;
  if ((e = launch_gather(c, idx, QUANT ? 1 : 0, sb.xg, nullptr, nullptr)) != cudaSuccess) return e;
  float* rep = c->buf.replicas;
  const int64_t rs = c->buf.replica_stride;
  const MomArgs mom = mom_args(c, c->replicas_equal_global);
  // forward
  for (int l = 1; l <= L; ++l) {
    const MlpLayer& ly = c->layers[l - 1];
    GemmArgs g{};
    g.A = l == 1 ? sb.xg : sb.z[l - 1]; g.a_batch = (int64_t)B * ly.in; g.a_m = ly.in; g.a_k = 1;
    g.B = rep + ly.w_off; g.b_batch = rs; g.b_n = ly.in; g.b_k = 1;
    g.M = B; g.N = ly.out; g.K = ly.in;
    g.C = sb.z[l]; g.c_batch = (int64_t)B * ly.out; g.c_m = ly.out;
    g.aux = rep + ly.b_off; g.aux_batch = rs; g.aux_m = 0;
    dim3 grid((ly.out + BN - 1) / BN, (B + BM - 1) / BM, P);
    prof_begin(c, MAVG_K_FWD);
    if (l == 1)
      k_simt_gemm<QUANT, LD_PLAIN, LD_PLAIN, true, true, EPI_FWD><<<grid, 256, 0, c->stream>>>(g);
    else
      k_simt_gemm<QUANT, LD_RELU, LD_PLAIN, true, true, EPI_FWD><<<grid, 256, 0, c->stream>>>(g);
    prof_end(c);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  // loss, dZ_L and the last bias
  const int C = cfg.dims[L];
  if ((e = launch_softmax_ce(c, sb.z[L], C, labels, losses + (step - 1), cfg.K, sb.dz[L], C,
                             nullptr, 0, nullptr, 0, true, mom)) != cudaSuccess)
    return e;
  // backward + SGD, layer L down to 1; dgrad reads W_l before wgrad overwrites it
  for (int l = L; l >= 1; --l) {
    const MlpLayer& ly = c->layers[l - 1];
    if (l > 1) {
      GemmArgs g{};
      g.A = sb.dz[l]; g.a_batch = (int64_t)B * ly.out; g.a_m = ly.out; g.a_k = 1;
      g.B = rep + ly.w_off; g.b_batch = rs; g.b_n = 1; g.b_k = ly.in;
      g.M = B; g.N = ly.in; g.K = ly.out;
      g.C = sb.dz[l - 1]; g.c_batch = (int64_t)B * ly.in; g.c_m = ly.in;
      g.aux = sb.z[l - 1]; g.aux_batch = (int64_t)B * ly.in; g.aux_m = ly.in;
      dim3 grid((ly.in + BN - 1) / BN, (B + BM - 1) / BM, P);
      prof_begin(c, MAVG_K_DGRAD);
      k_simt_gemm<QUANT, LD_PLAIN, LD_PLAIN, true, false, EPI_DGRAD><<<grid, 256, 0, c->stream>>>(g);
      prof_end(c);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    {
      GemmArgs g{};
      g.A = sb.dz[l]; g.a_batch = (int64_t)B * ly.out; g.a_m = 1; g.a_k = ly.out;
      g.B = l == 1 ? sb.xg : sb.z[l - 1]; g.b_batch = (int64_t)B * ly.in; g.b_n = 1; g.b_k = ly.in;
      g.M = ly.out; g.N = ly.in; g.K = B;
      g.C = rep + ly.w_off; g.c_batch = rs; g.c_m = ly.in;
      g.gamma = cfg.local_lr;
      g.mom = mom; g.u_off = ly.w_off;
      dim3 grid((ly.in + BN - 1) / BN, (ly.out + BM - 1) / BM, P);
      prof_begin(c, MAVG_K_WGRAD_SGD);
      if (l == 1)
        k_simt_gemm<QUANT, LD_PLAIN, LD_PLAIN, false, false, EPI_WGRAD_SGD><<<grid, 256, 0, c->stream>>>(g);
      else
        k_simt_gemm<QUANT, LD_PLAIN, LD_RELU, false, false, EPI_WGRAD_SGD><<<grid, 256, 0, c->stream>>>(g);
      prof_end(c);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (l < L) {
      dim3 grid((ly.out + 255) / 256, P);
      prof_begin(c, MAVG_K_WGRAD_SGD);
      k_simt_bias_sgd<<<grid, 256, 0, c->stream>>>(sb.dz[l], (int64_t)B * ly.out, B, ly.out, rep,
                                                   rs, ly.b_off, cfg.local_lr, mom);
      prof_end(c);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

}  // namespace

size_t simt_workspace_bytes(const mavg_config* cfg, size_t base, size_t* act_off) {
  *act_off = base;
  const size_t rows = (size_t)cfg->P * cfg->B;
  size_t off = base;
  auto take = [&](size_t floats) { off += (floats * sizeof(float) + 255) / 256 * 256; };
  take(rows * cfg->dims[0]);
  for (int l = 1; l <= cfg->n_layers; ++l) {
    take(rows * cfg->dims[l]);
    take(rows * cfg->dims[l]);
  }
  return off;
}

cudaError_t simt_step(mavg_ctx* c, int64_t round, int step) {
  return c->cfg.gemm_bf16 ? step_impl<true>(c, round, step) : step_impl<false>(c, round, step);
}

}  // namespace mavg
