// The structured mask step: unit scores (Lemma 1 and the two Wanda forms), the softmax-form sparsity allocation of
// Lemma 2 / Algorithm 1 Step 2, the exact top-k selection by radix select, and M (.) W.
#include <math.h>

#include <mutex>

#include "sp_common.cuh"

namespace sp {
namespace {

__device__ __forceinline__ float ld_f(const void* p, int32_t dt, int64_t i) {
  return dt == SP_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                       : reinterpret_cast<const float*>(p)[i];
}

__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  return v;
}

// Sum over the block in a fixed order; result valid in thread 0 and broadcast through smem[32].
__device__ double block_sum_bcast(double v, double* smem) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) smem[w] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double r = 0.0;
    const int nw = (blockDim.x + 31) >> 5;
    for (int i = 0; i < nw; ++i) r += smem[i];
    smem[32] = r;
  }
  __syncthreads();
  return smem[32];
}

__device__ double block_max_bcast(double v, double* smem) {
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_down_sync(0xffffffffu, v, o));
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) smem[w] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    double r = smem[0];
    const int nw = (blockDim.x + 31) >> 5;
    for (int i = 1; i < nw; ++i) r = fmax(r, smem[i]);
    smem[32] = r;
  }
  __syncthreads();
  return smem[32];
}

// ------------------------------------------------------------------------------------------------ Wanda scores
// partial column sums of W^2 (kind 0) or |W| (kind 1): grid (col blocks, row blocks) -> part[rb, cols]
__global__ void weight_col_partials_kernel(const float* __restrict__ W, int64_t rows, int64_t cols, int64_t ldw,
                                           int kind, int row_blocks, double* part) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  const int64_t rows_per = ceil_div(rows, (int64_t)row_blocks);
  const int64_t r0 = (int64_t)blockIdx.y * rows_per;
  const int64_t r1 = (r0 + rows_per < rows) ? r0 + rows_per : rows;
  double s = 0.0;
  for (int64_t r = r0; r < r1; ++r) {
    const double v = (double)W[r * ldw + c];
    s += kind == 0 ? v * v : fabs(v);
  }
  part[(int64_t)blockIdx.y * cols + c] = s;
}

__global__ void __launch_bounds__(1024) wanda_finish_kernel(const double* part, int row_blocks, int64_t cols,
                                                            int kind, int group, const float* colsq,
                                                            int64_t colsq_stride, const double* colabs,
                                                            double inv_tokens, int64_t n_units, float* scores,
                                                            double* importance) {
  __shared__ double sm[33];
  double acc = 0.0;
  for (int64_t u = threadIdx.x; u < n_units; u += blockDim.x) {
    double s = 0.0;
    for (int g = 0; g < group; ++g) {
      const int64_t j = u * group + g;
      double w = 0.0;
      for (int r = 0; r < row_blocks; ++r) w += part[(int64_t)r * cols + j];
      s += kind == 0 ? w * (double)colsq[j * colsq_stride] : w * colabs[j] * inv_tokens;
    }
    const float sc = (float)(kind == 0 ? sqrt(s) : s);
    scores[u] = sc;
    acc += (double)sc;
  }
  const double tot = block_sum_bcast(acc, sm);
  if (threadIdx.x == 0 && importance) importance[0] = tot / (double)n_units;
}

// ------------------------------------------------------------------------------------------------ Lemma 1
__global__ void lemma1_partials_kernel(sp_mat b, sp_mat c, sp_mat dd, sp_mat t, int64_t N, int64_t cols,
                                       int row_blocks, double* part) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= cols) return;
  const int64_t rows_per = ceil_div(N, (int64_t)row_blocks);
  const int64_t r0 = (int64_t)blockIdx.y * rows_per;
  const int64_t r1 = (r0 + rows_per < N) ? r0 + rows_per : N;
  double num = 0.0, den = 0.0;
  for (int64_t r = r0; r < r1; ++r) {
    const double vb = (double)ld_f(b.ptr, b.dtype, r * b.ld + j);
    const double vc = (double)ld_f(c.ptr, c.dtype, r * c.ld + j);
    const double vd = (double)ld_f(dd.ptr, dd.dtype, r * dd.ld + j);
    const double vt = (double)ld_f(t.ptr, t.dtype, r * t.ld + j);
    num += vc * vb + vd * vt;
    den += vc * vc + vd * vd;
  }
  part[((int64_t)blockIdx.y * cols + j) * 2 + 0] = num;
  part[((int64_t)blockIdx.y * cols + j) * 2 + 1] = den;
}

__global__ void __launch_bounds__(1024) lemma1_finish_kernel(const double* part, int row_blocks, int64_t cols,
                                                             int group, int64_t n_units, float* scores,
                                                             double* importance, double* relaxed, double r_layer,
                                                             double* unit_e) {
  __shared__ double sm[33];
  double acc_s = 0.0, acc_ie = 0.0;
  for (int64_t u = threadIdx.x; u < n_units; u += blockDim.x) {
    double num = 0.0, den = 0.0;
    for (int g = 0; g < group; ++g) {
      const int64_t j = u * group + g;
      for (int r = 0; r < row_blocks; ++r) {
        num += part[((int64_t)r * cols + j) * 2 + 0];
        den += part[((int64_t)r * cols + j) * 2 + 1];
      }
    }
    const double s = num / den;
    scores[u] = (float)s;
    unit_e[u * 2 + 0] = s;
    unit_e[u * 2 + 1] = den;
    acc_s += s;
    acc_ie += 1.0 / den;
  }
  const double sum_s = block_sum_bcast(acc_s, sm);
  const double sum_ie = block_sum_bcast(acc_ie, sm);
  if (threadIdx.x == 0 && importance) importance[0] = sum_s / (double)n_units;
  if (relaxed) {
    const double lam_half = (sum_s - r_layer * (double)n_units) / sum_ie;
    for (int64_t u = threadIdx.x; u < n_units; u += blockDim.x)
      relaxed[u] = unit_e[u * 2 + 0] - lam_half / unit_e[u * 2 + 1];
  }
}

// one warp per row j: cb = <T0[j], W1t[j]>, cc = <T0[j], W10[j]>; s = (cb + cc) / (2 cc)
__global__ void lemma1_gram_rows_kernel(const float* __restrict__ T0, const float* __restrict__ W1t,
                                        const float* __restrict__ W10, int64_t n, int64_t d, float* scores) {
  const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (j >= n) return;
  double cb = 0.0, cc = 0.0;
  for (int64_t q = lane; q < d; q += 32) {
    const double t0 = (double)T0[j * d + q];
    cb += t0 * (double)W1t[j * d + q];
    cc += t0 * (double)W10[j * d + q];
  }
  cb = warp_sum(cb);
  cc = warp_sum(cc);
  if (lane == 0) scores[j] = (float)((cb + cc) / (2.0 * cc));
}

__global__ void __launch_bounds__(1024) mean_scores_kernel(const float* scores, int64_t n, double* importance) {
  __shared__ double sm[33];
  double acc = 0.0;
  for (int64_t u = threadIdx.x; u < n; u += blockDim.x) acc += (double)scores[u];
  const double tot = block_sum_bcast(acc, sm);
  if (threadIdx.x == 0) importance[0] = tot / (double)n;
}

// ------------------------------------------------------------------------------------------------ allocation
__global__ void __launch_bounds__(1024) allocate_kernel(const double* I, const int64_t* n_units, int L, double rbar,
                                                        double T, int mode, double clip_hi, double* r_out,
                                                        int64_t* k_out) {
  __shared__ double sm[33];
  const int t = threadIdx.x;
  if (mode == SP_ALLOC_UNIFORM) {
    for (int l = t; l < L; l += blockDim.x) r_out[l] = rbar;
  } else {
    double mx = -INFINITY;
    for (int l = t; l < L; l += blockDim.x) mx = fmax(mx, -I[l] / T);
    mx = block_max_bcast(mx, sm);
    double s = 0.0;
    for (int l = t; l < L; l += blockDim.x) {
      const double w = exp(-I[l] / T - mx);
      r_out[l] = w;  // staged
      s += w;
    }
    const double wsum = block_sum_bcast(s, sm);
    if (mode == SP_ALLOC_SOFTMAX) {
      double clipped = 0.0, mu = 0.0;
      const double scale = rbar * (double)L;
      for (int l = t; l < L; l += blockDim.x) {
        const double raw = scale * (r_out[l] / wsum);
        if (raw > clip_hi) clipped = 1.0;
        const double r = fmin(fmax(raw, 0.0), clip_hi);
        r_out[l] = r;
        mu += r;
      }
      const double any = block_sum_bcast(clipped, sm);
      mu = block_sum_bcast(mu, sm) / (double)L;
      if (any == 0.0 && mu > 0.0) {
        const double f = rbar / mu;
        for (int l = t; l < L; l += blockDim.x) r_out[l] = fmin(fmax(r_out[l] * f, 0.0), clip_hi);
      }
    } else {  // inverse weighting
      double s1 = 0.0;
      for (int l = t; l < L; l += blockDim.x) {
        const double w = r_out[l] / wsum;
        r_out[l] = w;
        s1 += 1.0 - w;
      }
      const double inv = block_sum_bcast(s1, sm);
      const double scale = rbar * (double)L;
      for (int l = t; l < L; l += blockDim.x) {
        const double r = (L > 1) ? scale * (1.0 - r_out[l]) / inv : rbar;
        r_out[l] = fmin(fmax(r, 0.0), clip_hi);
      }
    }
  }
  __syncthreads();
  for (int l = t; l < L; l += blockDim.x) {
    const double nu = (double)n_units[l];
    k_out[l] = n_units[l] - (int64_t)floor(r_out[l] * nu + 0.5);
  }
}

// ------------------------------------------------------------------------------------------------ top-k
// Order-preserving key: larger float -> larger key; NaN is treated as -infinity, -0 as +0.
__device__ __forceinline__ uint32_t score_key(float v) {
  if (v != v) v = -INFINITY;
  uint32_t b = __float_as_uint(v);
  if ((b & 0x7fffffffu) == 0u) b = 0u;   // -0 and +0 are the same score
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// exclusive scan of a 0/1 flag over the block (1024 threads max); returns the exclusive prefix, total via *total
__device__ int block_excl_scan(int flag, int* warp_tot, int* total) {
  const int l = threadIdx.x & 31, w = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  const int within = __popc(bal & ((1u << l) - 1u));
  __syncthreads();
  if (l == 0) warp_tot[w] = __popc(bal);
  __syncthreads();
  int before = 0, tot = 0;
  const int nw = (blockDim.x + 31) >> 5;
  for (int i = 0; i < nw; ++i) {
    const int c = warp_tot[i];
    if (i < w) before += c;
    tot += c;
  }
  *total = tot;
  return before + within;
}

__global__ void __launch_bounds__(1024) topk_select_kernel(const float* __restrict__ scores, int64_t n, int64_t k,
                                                           uint8_t* mask, float* tau, int32_t* kept_idx) {
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_prefix;
  __shared__ int64_t s_krem;
  const int t = threadIdx.x;
  if (k <= 0 || k >= n) {
    for (int64_t i = t; i < n; i += blockDim.x) {
      mask[i] = k >= n ? 1 : 0;
      if (k >= n && kept_idx) kept_idx[i] = (int32_t)i;
    }
    if (t == 0 && tau) {
      float m = NAN;
      if (k >= n && n > 0) {  // smallest score
        uint32_t best = 0xffffffffu;
        for (int64_t i = 0; i < n; ++i) best = min(best, score_key(scores[i]));
        for (int64_t i = 0; i < n; ++i)
          if (score_key(scores[i]) == best) { m = scores[i]; break; }
      }
      tau[0] = m;
    }
    return;
  }
  if (t == 0) { s_prefix = 0u; s_krem = k; }
  __syncthreads();
  // find the key of the k-th largest score, 8 bits per pass from the top
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int i = t; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int64_t i = t; i < n; i += blockDim.x) {
      const uint32_t key = score_key(scores[i]);
      if ((key & hi_mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xffu], 1);
    }
    __syncthreads();
    if (t == 0) {
      int64_t rem = s_krem;
      int bin = 255;
      for (; bin > 0; --bin) {
        if (hist[bin] >= rem) break;
        rem -= hist[bin];
      }
      s_krem = rem;  // how many to take from this bin
      s_prefix = prefix | ((uint32_t)bin << shift);
    }
    __syncthreads();
  }
  const uint32_t tkey = s_prefix;
  const int64_t take_eq = s_krem;  // ties at the threshold that are kept (lowest indices first)
  int64_t eq_before = 0, kept_before = 0;
  bool tau_written = false;
  for (int64_t base = 0; base < n; base += blockDim.x) {
    const int64_t i = base + t;
    uint32_t key = 0;
    const bool valid = i < n;
    if (valid) key = score_key(scores[i]);
    const int is_eq = valid && key == tkey;
    int tot_eq, tot_keep;
    const int eq_rank = block_excl_scan(is_eq, warp_tot, &tot_eq);
    const int keep = valid && (key > tkey || (is_eq && eq_before + eq_rank < take_eq));
    const int keep_rank = block_excl_scan(keep, warp_tot, &tot_keep);
    if (valid) {
      mask[i] = (uint8_t)keep;
      if (keep && kept_idx) kept_idx[kept_before + keep_rank] = (int32_t)i;
      if (is_eq && !tau_written && tau && eq_before + eq_rank == 0) tau[0] = scores[i] != scores[i] ? -INFINITY : scores[i];
    }
    eq_before += tot_eq;
    kept_before += tot_keep;
    if (eq_before > 0) tau_written = true;
  }
}

__global__ void __launch_bounds__(1024) mask_to_index_kernel(const uint8_t* mask, int64_t n, int32_t* kept_idx) {
  __shared__ int warp_tot[32];
  int64_t before = 0;
  for (int64_t base = 0; base < n; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    const int keep = (i < n) && mask[i] != 0;
    int tot;
    const int rank = block_excl_scan(keep, warp_tot, &tot);
    if (keep) kept_idx[before + rank] = (int32_t)i;
    before += tot;
  }
}

__global__ void zero_rows_kernel(const uint8_t* mask, int group, float* W, int64_t rows, int64_t cols, int64_t ld) {
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    if (!mask[i / group]) W[i * ld + j] = 0.f;
  }
}

__global__ void zero_cols_kernel(const uint8_t* mask, int group, float* W, int64_t rows, int64_t cols, int64_t ld) {
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    if (!mask[j / group]) W[i * ld + j] = 0.f;
  }
}

__global__ void mask_rows_copy_kernel(const uint8_t* mask, const float* src, int64_t lds, float* dst, int64_t ldd,
                                      int64_t rows, int64_t cols) {
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    dst[i * ldd + j] = mask[i] ? src[i * lds + j] : 0.f;
  }
}

inline int grid_for(int64_t total, int threads) {
  int64_t b = ceil_div(total, (int64_t)threads);
  if (b > 148 * 16) b = 148 * 16;
  if (b < 1) b = 1;
  return (int)b;
}

inline int row_blocks_for(int64_t rows, int64_t cols) {
  const int64_t cb = ceil_div(cols, 256);
  int64_t rb = ceil_div(148 * 4, cb);
  if (rb > rows) rb = rows;
  if (rb < 1) rb = 1;
  return (int)rb;
}

}  // namespace

int score_row_blocks(int64_t rows, int64_t cols) { return row_blocks_for(rows, cols); }

cudaError_t wanda_scores(int kind, int group, const float* W, int64_t rows, int64_t ldw, const float* colsq,
                         int64_t colsq_stride, const double* colabs, double inv_tokens, int64_t n_units,
                         float* scores, double* importance, double* scratch, cudaStream_t stream) {
  const int64_t cols = n_units * group;
  if (cols == 0) return cudaSuccess;
  const int rb = row_blocks_for(rows, cols);
  const int k = kind == SP_SCORE_WANDA_L2 ? 0 : 1;
  ProfScope prof(PK_SCORES, 0.0, (double)rows * (double)cols * 4.0, stream);
  count_launch();
  weight_col_partials_kernel<<<dim3((unsigned)ceil_div(cols, 256), (unsigned)rb), 256, 0, stream>>>(W, rows, cols, ldw,
                                                                                                   k, rb, scratch);
  count_launch();
  wanda_finish_kernel<<<1, 1024, 0, stream>>>(scratch, rb, cols, k, group, colsq, colsq_stride, colabs, inv_tokens,
                                              n_units, scores, importance);
  return cudaGetLastError();
}

cudaError_t lemma1_scores_stream(const sp_mat& b, const sp_mat& c, const sp_mat& dd, const sp_mat& t, int group,
                                 int64_t n_units, float* scores, double* importance, double* relaxed, double r_layer,
                                 double* scratch, cudaStream_t stream) {
  const int64_t cols = n_units * group;
  const int64_t N = b.rows;
  if (cols == 0) return cudaSuccess;
  const int rb = row_blocks_for(N, cols);
  double* part = scratch;
  double* unit_e = scratch + (size_t)rb * cols * 2;
  ProfScope prof(PK_SCORES, 0.0, (double)N * (double)cols * (double)(dtype_size(b.dtype) + dtype_size(c.dtype) +
                                                                    dtype_size(dd.dtype) + dtype_size(t.dtype)),
                 stream);
  count_launch();
  lemma1_partials_kernel<<<dim3((unsigned)ceil_div(cols, 256), (unsigned)rb), 256, 0, stream>>>(b, c, dd, t, N, cols,
                                                                                               rb, part);
  count_launch();
  lemma1_finish_kernel<<<1, 1024, 0, stream>>>(part, rb, cols, group, n_units, scores, importance, relaxed, r_layer,
                                               unit_e);
  return cudaGetLastError();
}

cudaError_t lemma1_scores_gram(const float* T0, const float* W1t, const float* W10, int64_t n, int64_t d,
                               float* scores, double* importance, double* scratch, cudaStream_t stream) {
  (void)scratch;
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_SCORES, 0.0, (double)n * (double)d * 12.0, stream);
  count_launch();
  lemma1_gram_rows_kernel<<<(unsigned)ceil_div(n * 32, 256), 256, 0, stream>>>(T0, W1t, W10, n, d, scores);
  count_launch();
  mean_scores_kernel<<<1, 1024, 0, stream>>>(scores, n, importance);
  return cudaGetLastError();
}

cudaError_t allocate_sparsity(const double* I, const int64_t* n_units, int L, double rbar, double T, int mode,
                              double clip_hi, double* r_out, int64_t* k_out, cudaStream_t stream) {
  ProfScope prof(PK_ALLOCATE, 0.0, (double)L * 32.0, stream);
  count_launch();
  allocate_kernel<<<1, 1024, 0, stream>>>(I, n_units, L, rbar, T, mode, clip_hi, r_out, k_out);
  return cudaGetLastError();
}

cudaError_t topk_select(const float* scores, int64_t n, int64_t k, uint8_t* mask, float* tau, int32_t* kept_idx,
                        cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_TOPK, 0.0, (double)n * 5.0, stream);
  count_launch();
  topk_select_kernel<<<1, 1024, 0, stream>>>(scores, n, k, mask, tau, kept_idx);
  return cudaGetLastError();
}

cudaError_t mask_to_index(const uint8_t* mask, int64_t n, int32_t* kept_idx, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  count_launch();
  mask_to_index_kernel<<<1, 1024, 0, stream>>>(mask, n, kept_idx);
  return cudaGetLastError();
}

cudaError_t zero_pruned(const uint8_t* mask, int group, float* W_rows, int64_t r_rows, int64_t r_cols, int64_t r_ld,
                        float* W_cols, int64_t c_rows, int64_t c_cols, int64_t c_ld, cudaStream_t stream) {
  if (W_rows && r_rows * r_cols > 0) {
    ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
    count_launch();
    zero_rows_kernel<<<grid_for(r_rows * r_cols, 256), 256, 0, stream>>>(mask, group, W_rows, r_rows, r_cols, r_ld);
  }
  if (W_cols && c_rows * c_cols > 0) {
    count_launch();
    zero_cols_kernel<<<grid_for(c_rows * c_cols, 256), 256, 0, stream>>>(mask, group, W_cols, c_rows, c_cols, c_ld);
  }
  return cudaGetLastError();
}

cudaError_t mask_rows_copy(const uint8_t* mask, const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows,
                           int64_t cols, cudaStream_t stream) {
  if (rows * cols == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  mask_rows_copy_kernel<<<grid_for(rows * cols, 256), 256, 0, stream>>>(mask, src, lds, dst, ldd, rows, cols);
  return cudaGetLastError();
}

}  // namespace sp

// ------------------------------------------------------------------------------------ static-scratch score entry
// Wanda scores for callers that hold no workspace and must not allocate one.  The partial column sums live in a
// file-scope device array that every GPU loading the library carries until the process exits.
namespace {

constexpr size_t kStaticScratchDoubles = (size_t)1 << 18;   // 2 MiB
static __device__ __align__(256) double g_static_scratch[kStaticScratchDoubles];

constexpr int kMaxDevices = 64;
double* g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mutex;

// Device address of g_static_scratch on the current device.  In host code the array's name is only a handle, so the
// address is looked up once per device (with that device current) and cached.
sp_status static_scratch_address(double** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return SP_ERR_CUDA;
    g_static_scratch_addr[dev] = reinterpret_cast<double*>(p);
  }
  *out = g_static_scratch_addr[dev];
  return SP_OK;
}

}  // namespace

extern "C" sp_status sp_struct_scores_static(int32_t kind, int32_t group, const sp_score_inputs* in, int64_t n_units,
                                             float* scores, double* layer_importance, void* stream) {
  if (!in || !scores) return SP_ERR_INVALID_ARG;
  if (kind != SP_SCORE_WANDA_L2 && kind != SP_SCORE_WANDA_L1) return SP_ERR_UNSUPPORTED;
  if (group < 1 || n_units < 1) return SP_ERR_SHAPE;
  if (n_units > SP_STATIC_SCORES_MAX_COLS / group) return SP_ERR_STATIC_LIMIT;
  const int64_t cols = n_units * group;
  if (!in->W.ptr) return SP_ERR_INVALID_ARG;
  if (in->W.dtype != SP_F32) return SP_ERR_DTYPE;
  if (in->W.cols != cols || in->W.ld < cols || in->W.rows < 1) return SP_ERR_SHAPE;
  if (kind == SP_SCORE_WANDA_L2 && (!in->colsq || in->colsq_stride < 1)) return SP_ERR_INVALID_ARG;
  if (kind == SP_SCORE_WANDA_L1 && !in->colabs) return SP_ERR_INVALID_ARG;
  // the partial sums take row_blocks x cols doubles; row_blocks shrinks as cols grows, so the product stays bounded
  if ((size_t)sp::score_row_blocks(in->W.rows, cols) * (size_t)cols > kStaticScratchDoubles)
    return SP_ERR_STATIC_LIMIT;
  double* scratch = nullptr;
  const sp_status st = static_scratch_address(&scratch);
  if (st != SP_OK) return st;
  // every partial sum that the finishing kernel reads is written by the first kernel of this same call, so nothing
  // left behind by an earlier call is ever read and no clearing is needed
  if (sp::wanda_scores(kind, group, reinterpret_cast<const float*>(in->W.ptr), in->W.rows, in->W.ld, in->colsq,
                       in->colsq_stride, in->colabs, in->inv_tokens, n_units, scores, layer_importance, scratch,
                       reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SP_ERR_CUDA;
  return SP_OK;
}
