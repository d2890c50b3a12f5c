// Elementwise and row-wise kernels of the multi-head-attention auxiliary updates (Appendix A, "Computation on
// Multi-Head Attention layers", Method 2; Algorithm 2, SparseLLM2).  The contractions around them (logits, P V, the
// gradient products) are batched tensor-core GEMMs issued by the host code in sp_api.cu; everything here is bound by
// memory bandwidth: one warp per row of a [pairs, T, T] tensor, 16-byte accesses where the layout allows.
#include "sp_common.cuh"

namespace sp {
namespace {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

constexpr int kRowWarps = 8;

// S[row, :] <- softmax over the keys of the row (in place).  rows = pairs * T; row r belongs to query t = r % T; with
// `causal` keys u > t get probability 0.  Optional bf16 copy.
__global__ void __launch_bounds__(kRowWarps * 32) softmax_rows_kernel(float* __restrict__ S, int64_t rows, int T,
                                                                      int causal, __nv_bfloat16* __restrict__ Sb,
                                                                      int64_t plane) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * kRowWarps + (threadIdx.x >> 5);
  if (r >= rows) return;
  float* row = S + r * T;
  const int lim = causal ? (int)(r % T) + 1 : T;
  float mx = -INFINITY;
  for (int u = lane; u < lim; u += 32) mx = fmaxf(mx, row[u]);
  mx = warp_max(mx);
  float sum = 0.f;
  for (int u = lane; u < lim; u += 32) sum += __expf(row[u] - mx);
  sum = warp_sum(sum);
  const float inv = 1.f / sum;
  for (int u = lane; u < T; u += 32) {
    const float v = u < lim ? __expf(row[u] - mx) * inv : 0.f;
    row[u] = v;
    if (Sb) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(v);
      Sb[r * T + u] = hi;
      if (plane > 0) Sb[plane + r * T + u] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
  }
}

// Gradient step of Eq. (85) on the attention probabilities of every (sequence, head) pair:
//   P <- P - eta_b (-2 alpha G1 + 2 beta (P - Phi)),  G1 = R V^T from the preceding product, eta_b per pair.
__global__ void __launch_bounds__(256) p_update_kernel(float* __restrict__ P, const float* __restrict__ Phi,
                                                       const float* __restrict__ G1, const float* __restrict__ eta,
                                                       int64_t per_pair, int64_t total, float alpha, float beta,
                                                       __nv_bfloat16* __restrict__ Pb, int64_t plane) {
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const float et = eta[e / per_pair];
    const float p = P[e];
    const float g = -2.f * alpha * G1[e] + 2.f * beta * (p - Phi[e]);
    const float pn = p - et * g;
    P[e] = pn;
    if (Pb) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(pn);
      Pb[e] = hi;
      if (plane > 0) Pb[plane + e] = __float2bfloat16_rn(pn - __bfloat162float(hi));
    }
  }
}

// Softmax and its backward for the softmax term of Eq. (87), one warp per row of logits S:
//   Phi = softmax(S),  E = Phi - P,  dS = 2 beta Phi (E - sum_u E Phi)  -> fp32 in place of S and / or bf16 copy.
__global__ void __launch_bounds__(kRowWarps * 32) softmax_backward_rows_kernel(float* __restrict__ S,
                                                                               const float* __restrict__ P,
                                                                               int64_t rows, int T, int causal,
                                                                               float beta,
                                                                               __nv_bfloat16* __restrict__ dSb) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * kRowWarps + (threadIdx.x >> 5);
  if (r >= rows) return;
  float* row = S + r * T;
  const float* prow = P + r * T;
  const int lim = causal ? (int)(r % T) + 1 : T;
  float mx = -INFINITY;
  for (int u = lane; u < lim; u += 32) mx = fmaxf(mx, row[u]);
  mx = warp_max(mx);
  float sum = 0.f;
  for (int u = lane; u < lim; u += 32) sum += __expf(row[u] - mx);
  sum = warp_sum(sum);
  const float inv = 1.f / sum;
  float dot = 0.f;        // sum_u E Phi (Phi = 0 beyond the causal limit)
  for (int u = lane; u < lim; u += 32) {
    const float ph = __expf(row[u] - mx) * inv;
    dot = fmaf(ph - prow[u], ph, dot);
  }
  dot = warp_sum(dot);
  for (int u = lane; u < T; u += 32) {
    float v = 0.f;
    if (u < lim) {
      const float ph = __expf(row[u] - mx) * inv;
      v = 2.f * beta * ph * (ph - prow[u] - dot);
    }
    row[u] = v;
    if (dSb) dSb[r * T + u] = __float2bfloat16_rn(v);
  }
}

// Sum of squares of the [T, d_h] slice of every (sequence, head) pair of up to two token-major [tokens, d] tensors;
// one block per pair, fixed summation order.  out[b] = sum x^2 (+ sum y^2), b = seq * H + head.
__global__ void __launch_bounds__(256) pair_sumsq_kernel(const float* __restrict__ x, const float* __restrict__ y,
                                                         int64_t ld, int T, int d_h, int H, double* __restrict__ out) {
  __shared__ double sm[256];
  const int b = blockIdx.x, seq = b / H, head = b % H;
  const int64_t base = (int64_t)seq * T * ld + (int64_t)head * d_h;
  double acc = 0.0;
  const int total = T * d_h;
  for (int e = threadIdx.x; e < total; e += 256) {
    const int64_t o = base + (int64_t)(e / d_h) * ld + (e % d_h);
    const float v = x[o];
    acc += (double)v * v;
    if (y) {
      const float w = y[o];
      acc += (double)w * w;
    }
  }
  sm[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[b] = sm[0];
}

// Step sizes from the sums above: mode 0 (Eq. 85): eta = 1 / (2 (alpha s + beta));
// mode 1 (Eq. 87): eta = eta_z / (2 alpha + beta s / d_h).
__global__ void step_size_kernel(const double* __restrict__ s, int n, int mode, double alpha, double beta, double eta_z,
                                 int d_h, float* __restrict__ eta) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n) return;
  eta[b] = mode == 0 ? (float)(1.0 / (2.0 * (alpha * s[b] + beta)))
                     : (float)(eta_z / (2.0 * alpha + beta * s[b] / (double)d_h));
}

// Gradient step of Eq. (87) on the projection outputs, token-major [tokens, d]:
//   Z <- Z - eta_b (G + 2 alpha (Z - Tg)) for Z in {Zq, Zk}, b = (token / T) * H + column / d_h;
// optional bf16 hi / lo planes of the new values (operands of the next logits product).
__global__ void __launch_bounds__(256) z_update_kernel(float* __restrict__ Zq, float* __restrict__ Zk,
                                                       const float* __restrict__ Gq, const float* __restrict__ Gk,
                                                       const float* __restrict__ Tq, const float* __restrict__ Tk,
                                                       const float* __restrict__ eta, int64_t tokens, int d, int T,
                                                       int d_h, float alpha, __nv_bfloat16* __restrict__ Zqs,
                                                       __nv_bfloat16* __restrict__ Zks, int64_t plane) {
  const int H = d / d_h;
  const int64_t total = tokens * d;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t tok = e / d;
    const int c = (int)(e % d);
    const float et = eta[(tok / T) * H + c / d_h];
    const float zq = Zq[e], zk = Zk[e];
    const float nq = zq - et * (Gq[e] + 2.f * alpha * (zq - Tq[e]));
    const float nk = zk - et * (Gk[e] + 2.f * alpha * (zk - Tk[e]));
    Zq[e] = nq;
    Zk[e] = nk;
    if (Zqs) {
      const __nv_bfloat16 hq = __float2bfloat16_rn(nq), hk = __float2bfloat16_rn(nk);
      Zqs[e] = hq;
      Zqs[plane + e] = __float2bfloat16_rn(nq - __bfloat162float(hq));
      Zks[e] = hk;
      Zks[plane + e] = __float2bfloat16_rn(nk - __bfloat162float(hk));
    }
  }
}

// hi / lo bf16 planes of a dense fp32 tensor of `total` elements: dst[e] = bf16(x), dst[plane + e] = bf16(x - hi).
__global__ void __launch_bounds__(256) split_planes_kernel(const float* __restrict__ x, int64_t total,
                                                           __nv_bfloat16* __restrict__ dst, int64_t plane) {
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const float v = x[e];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    dst[e] = hi;
    if (plane > 0) dst[plane + e] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

__global__ void set_identity_kernel(float* A, int64_t n, int64_t ld) {
  const int64_t total = n * n;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / n, j = e % n;
    A[i * ld + j] = i == j ? 1.f : 0.f;
  }
}

unsigned grid_1d(int64_t total, int threads) {
  int64_t b = (total + threads - 1) / threads;
  const int64_t cap = (int64_t)sm_count() * 16;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (unsigned)b;
}

}  // namespace

cudaError_t mha_softmax_rows(float* S, int64_t pairs, int T, bool causal, void* Sb, int64_t plane,
                             cudaStream_t stream) {
  const int64_t rows = pairs * T;
  if (rows == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)rows * T * 8.0, stream);
  count_launch();
  softmax_rows_kernel<<<(unsigned)ceil_div(rows, (int64_t)kRowWarps), kRowWarps * 32, 0, stream>>>(
      S, rows, T, causal ? 1 : 0, reinterpret_cast<__nv_bfloat16*>(Sb), plane);
  return cudaGetLastError();
}

cudaError_t mha_p_update(float* P, const float* Phi, const float* G1, const float* eta, int64_t pairs, int T,
                         double alpha, double beta, void* Pb, int64_t plane, cudaStream_t stream) {
  const int64_t total = pairs * T * T;
  if (total == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)total * 16.0, stream);
  count_launch();
  p_update_kernel<<<grid_1d(total, 256), 256, 0, stream>>>(P, Phi, G1, eta, (int64_t)T * T, total, (float)alpha,
                                                           (float)beta, reinterpret_cast<__nv_bfloat16*>(Pb), plane);
  return cudaGetLastError();
}

cudaError_t mha_softmax_backward_rows(float* S, const float* P, int64_t pairs, int T, bool causal, double beta,
                                      void* dSb, cudaStream_t stream) {
  const int64_t rows = pairs * T;
  if (rows == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)rows * T * 12.0, stream);
  count_launch();
  softmax_backward_rows_kernel<<<(unsigned)ceil_div(rows, (int64_t)kRowWarps), kRowWarps * 32, 0, stream>>>(
      S, P, rows, T, causal ? 1 : 0, (float)beta, reinterpret_cast<__nv_bfloat16*>(dSb));
  return cudaGetLastError();
}

cudaError_t mha_step_sizes(const float* x, const float* y, int64_t ld, int64_t n_seq, int T, int d_h, int H, int mode,
                           double alpha, double beta, double eta_z, double* sums, float* eta, cudaStream_t stream) {
  const int n = (int)(n_seq * H);
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch(2);
  pair_sumsq_kernel<<<n, 256, 0, stream>>>(x, y, ld, T, d_h, H, sums);
  step_size_kernel<<<(n + 255) / 256, 256, 0, stream>>>(sums, n, mode, alpha, beta, eta_z, d_h, eta);
  return cudaGetLastError();
}

cudaError_t mha_z_update(float* Zq, float* Zk, const float* Gq, const float* Gk, const float* Tq, const float* Tk,
                         const float* eta, int64_t tokens, int d, int T, int d_h, double alpha, void* Zqs, void* Zks,
                         int64_t plane, cudaStream_t stream) {
  const int64_t total = tokens * d;
  if (total == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)total * 32.0, stream);
  count_launch();
  z_update_kernel<<<grid_1d(total, 256), 256, 0, stream>>>(Zq, Zk, Gq, Gk, Tq, Tk, eta, tokens, d, T, d_h, (float)alpha,
                                                           reinterpret_cast<__nv_bfloat16*>(Zqs),
                                                           reinterpret_cast<__nv_bfloat16*>(Zks), plane);
  return cudaGetLastError();
}

cudaError_t set_identity(float* A, int64_t n, int64_t ld, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  count_launch();
  set_identity_kernel<<<grid_1d(n * n, 256), 256, 0, stream>>>(A, n, ld);
  return cudaGetLastError();
}

cudaError_t split_planes(const float* x, int64_t total, void* dst, int64_t plane, cudaStream_t stream) {
  if (total == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)total * 8.0, stream);
  count_launch();
  split_planes_kernel<<<grid_1d(total, 256), 256, 0, stream>>>(x, total, reinterpret_cast<__nv_bfloat16*>(dst), plane);
  return cudaGetLastError();
}

}  // namespace sp
