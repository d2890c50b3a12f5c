// The structured mask step: unit scores (Lemma 1 and the two Wanda forms), the softmax-form sparsity allocation of
// Lemma 2 / Algorithm 1 Step 2, the exact top-k selection by radix select, and M (.) W.
#include <math.h>

#include <algorithm>
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
// s_u = sqrt(sum_{j in unit u} |W[:, j]|_2^2 * colsq[j])  (L2 form)  or  sum_j |W[:, j]|_1 * colabs[j] / tokens  (L1 form),
// and the layer importance mean_u s_u, in ONE launch that reads W once.
//   grid (column groups of 128, row blocks); a lane owns 4 adjacent columns (one 16-byte load per row), the 8 warps of a
//   block take every 8th row of the block's row range, 8 rows of loads in flight per thread.
//   stage 1: every block writes its 128 partial column sums (fp64, fixed order) to part[row block][col];
//   stage 2: the block that arrives last at its column group's ticket adds the row blocks' partials in order; when
//            units do not straddle column groups (128 % group == 0) it writes their scores and the sum of them,
//            else the finished per-column values;
//   stage 3: the block that arrives last at the final ticket adds the groups' sums (or first turns column values
//            into unit scores) and writes the mean.
// Which block is last varies; what it adds, and in which order, does not: the result is deterministic.
// tickets[0 .. gridDim.x] must be zero at launch; each is set back to zero by the block that consumed it.
constexpr int kWsCols = 128, kWsWarps = 8, kWsUnroll = 8;

__global__ void __launch_bounds__(kWsWarps * 32) wanda_scores_kernel(
    const float* __restrict__ W, int64_t rows, int64_t cols, int64_t ldw, int vec_ok, int kind, int group,
    const float* __restrict__ colsq, int64_t colsq_stride, const double* __restrict__ colabs, double inv_tokens,
    int64_t n_units, float* scores, double* importance, double* part, double* colval, unsigned int* tickets) {
  __shared__ double red[kWsWarps][kWsCols];
  __shared__ double sm[33];
  __shared__ int s_last;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int row_blocks = (int)gridDim.y;
  const int64_t c0 = (int64_t)blockIdx.x * kWsCols + 4 * lane;
  const int64_t rows_per = ceil_div(rows, (int64_t)row_blocks);
  const int64_t r0 = (int64_t)blockIdx.y * rows_per;
  const int64_t r1 = (r0 + rows_per < rows) ? r0 + rows_per : rows;
  const bool full = vec_ok && c0 + 3 < cols;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  for (int64_t rb = r0 + warp; rb < r1; rb += (int64_t)kWsWarps * kWsUnroll) {
    float4 v[kWsUnroll];
#pragma unroll
    for (int q = 0; q < kWsUnroll; ++q) {
      const int64_t r = rb + (int64_t)q * kWsWarps;
      v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < r1) {
        const float* src = W + r * ldw + c0;
        if (full) {
          v[q] = *reinterpret_cast<const float4*>(src);
        } else {
          if (c0 < cols) v[q].x = src[0];
          if (c0 + 1 < cols) v[q].y = src[1];
          if (c0 + 2 < cols) v[q].z = src[2];
          if (c0 + 3 < cols) v[q].w = src[3];
        }
      }
    }
#pragma unroll
    for (int q = 0; q < kWsUnroll; ++q) {
      const double x = v[q].x, y = v[q].y, z = v[q].z, w = v[q].w;
      if (kind == 0) {
        acc[0] = fma(x, x, acc[0]); acc[1] = fma(y, y, acc[1]); acc[2] = fma(z, z, acc[2]); acc[3] = fma(w, w, acc[3]);
      } else {
        acc[0] += fabs(x); acc[1] += fabs(y); acc[2] += fabs(z); acc[3] += fabs(w);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) red[warp][4 * lane + j] = acc[j];
  __syncthreads();
  if (t < kWsCols) {
    const int64_t c = (int64_t)blockIdx.x * kWsCols + t;
    if (c < cols) {
      double sum = 0.0;
#pragma unroll
      for (int w = 0; w < kWsWarps; ++w) sum += red[w][t];
      part[(int64_t)blockIdx.y * cols + c] = sum;
    }
  }
  // ---- stage 2: last block of this column group
  __threadfence();
  __syncthreads();
  if (t == 0) s_last = atomicAdd(&tickets[blockIdx.x], 1u) == (unsigned)(row_blocks - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // units that lie inside one column group are finished here; otherwise stage 3 adds column values across groups
  const bool direct = (kWsCols % group) == 0;
  double* cv = &red[0][0];
  if (t < kWsCols) {
    const int64_t c = (int64_t)blockIdx.x * kWsCols + t;
    double val = 0.0;
    if (c < cols) {
      double w = 0.0;
      int r = 0;
      for (; r + 8 <= row_blocks; r += 8) {          // independent loads, added in order
        double pv[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) pv[q] = __ldcg(&part[(int64_t)(r + q) * cols + c]);
#pragma unroll
        for (int q = 0; q < 8; ++q) w += pv[q];
      }
      for (; r < row_blocks; ++r) w += __ldcg(&part[(int64_t)r * cols + c]);
      val = kind == 0 ? w * (double)colsq[c * colsq_stride] : w * colabs[c] * inv_tokens;
      if (!direct) colval[c] = val;
    }
    cv[t] = val;
  }
  __syncthreads();
  if (direct) {
    const int upg = kWsCols / group;                  // units per column group
    double mine = 0.0;
    if (t < upg) {
      const int64_t u = (int64_t)blockIdx.x * upg + t;
      if (u < n_units) {
        double sc = 0.0;
        for (int g = 0; g < group; ++g) sc += cv[t * group + g];
        const float f = (float)(kind == 0 ? sqrt(sc) : sc);
        scores[u] = f;
        mine = (double)f;
      }
    }
    mine = block_sum_bcast(mine, sm);
    if (t == 0) colval[blockIdx.x] = mine;            // sum of this group's scores
  }
  // ---- stage 3: last column group
  __threadfence();
  __syncthreads();
  if (t == 0) {
    tickets[blockIdx.x] = 0u;
    s_last = atomicAdd(&tickets[gridDim.x], 1u) == gridDim.x - 1u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  double tot = 0.0;
  if (direct) {
    for (int64_t gq = t; gq < (int64_t)gridDim.x; gq += blockDim.x) tot += __ldcg(&colval[gq]);
  } else {
    for (int64_t u0 = 0; u0 < n_units; u0 += (int64_t)blockDim.x * 4) {
      double sc[4] = {0.0, 0.0, 0.0, 0.0};
      for (int g = 0; g < group; ++g) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int64_t u = u0 + (int64_t)q * blockDim.x + t;
          if (u < n_units) sc[q] += __ldcg(&colval[u * group + g]);
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t u = u0 + (int64_t)q * blockDim.x + t;
        if (u < n_units) {
          const float f = (float)(kind == 0 ? sqrt(sc[q]) : sc[q]);
          scores[u] = f;
          tot += (double)f;
        }
      }
    }
  }
  tot = block_sum_bcast(tot, sm);
  if (t == 0) {
    if (importance) importance[0] = tot / (double)n_units;
    tickets[gridDim.x] = 0u;
  }
}

// ------------------------------------------------------------------------------------------------ weight statistics
// Sums {|w|, w, w^2} over rectangular slices of a weight matrix (Algorithm "-distribute", Step 1).
//   grid (blocks, parts): block b is the rectangle rows [r0, r1) x columns [c0, c1); its rows are cut into `parts`
//   ranges, one CTA each.  Threads walk the CTA's range row-major in 16-byte pieces (scalars when the slice is not
//   16-byte aligned), eight loads in flight each; fp32 sums over the 32 or 64 values of a round, fp64 running sums,
//   fixed-order block reduction -> part[b][p][3].
template <typename T>
struct StatVec;
template <>
struct StatVec<float> {
  static constexpr int V = 4;
  typedef float4 Raw;
  __device__ static Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ static float get(const Raw& v, int j) { return j == 0 ? v.x : j == 1 ? v.y : j == 2 ? v.z : v.w; }
};
template <>
struct StatVec<__nv_bfloat16> {
  static constexpr int V = 8;
  typedef uint4 Raw;
  __device__ static Raw zero() { return make_uint4(0u, 0u, 0u, 0u); }
  __device__ static float get(const Raw& v, int j) {
    const uint32_t w = (j >> 1) == 0 ? v.x : (j >> 1) == 1 ? v.y : (j >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16));
  }
};
__device__ __forceinline__ float stat_scalar(const float* p) { return *p; }
__device__ __forceinline__ float stat_scalar(const __nv_bfloat16* p) { return __bfloat162float(*p); }

constexpr int kStatInFlight = 8;     // 16-byte loads a thread keeps in flight

template <typename T>
__global__ void __launch_bounds__(256, 4) weight_stats_partial_kernel(const T* __restrict__ W, int64_t ld,
                                                                      int64_t rows, int64_t cols, int axis,
                                                                      int64_t group, int vec_ok, double* part) {
  typedef typename StatVec<T>::Raw Raw;
  constexpr int V = StatVec<T>::V;
  __shared__ double sm[33];
  const int64_t b = blockIdx.x;
  const int parts = (int)gridDim.y;
  int64_t r0 = 0, r1 = rows, c0 = 0, c1 = cols;
  if (group > 0) {
    if (axis == 0) { r0 = b * group; r1 = r0 + group; }
    else { c0 = b * group; c1 = c0 + group; }
  }
  const int64_t rows_per = ceil_div(r1 - r0, (int64_t)parts);
  const int64_t pr0 = r0 + (int64_t)blockIdx.y * rows_per;
  const int64_t pr1 = (pr0 + rows_per < r1) ? pr0 + rows_per : r1;
  const int64_t width = c1 - c0;
  double s_abs = 0.0, s_sum = 0.0, s_sq = 0.0;
  if (pr0 < pr1) {
    if (vec_ok && width % V == 0) {
      const int64_t nq = width / V, total = (pr1 - pr0) * nq;
      for (int64_t e0 = threadIdx.x; e0 < total; e0 += (int64_t)blockDim.x * kStatInFlight) {
        Raw raw[kStatInFlight];
#pragma unroll
        for (int q = 0; q < kStatInFlight; ++q) {
          const int64_t e = e0 + (int64_t)q * blockDim.x;
          raw[q] = e < total ? *reinterpret_cast<const Raw*>(W + (pr0 + e / nq) * ld + c0 + (e % nq) * V)
                             : StatVec<T>::zero();
        }
        // the values of this round are summed in fp32 (32 or 64 terms), the running sums are fp64: the fp64 pipe is
        // narrow, and one conversion per value would make this kernel compute-bound
        float fa = 0.f, fs = 0.f, fq = 0.f;
#pragma unroll
        for (int q = 0; q < kStatInFlight; ++q)
#pragma unroll
          for (int j = 0; j < V; ++j) {
            const float x = StatVec<T>::get(raw[q], j);
            fa += fabsf(x);
            fs += x;
            fq = fmaf(x, x, fq);
          }
        s_abs += (double)fa;
        s_sum += (double)fs;
        s_sq += (double)fq;
      }
    } else {
      const int64_t total = (pr1 - pr0) * width;
      for (int64_t e = threadIdx.x; e < total; e += blockDim.x) {
        const double x = (double)stat_scalar(W + (pr0 + e / width) * ld + c0 + e % width);
        s_abs += fabs(x);
        s_sum += x;
        s_sq = fma(x, x, s_sq);
      }
    }
  }
  s_abs = block_sum_bcast(s_abs, sm);
  s_sum = block_sum_bcast(s_sum, sm);
  s_sq = block_sum_bcast(s_sq, sm);
  if (threadIdx.x == 0) {
    double* o = part + (b * parts + blockIdx.y) * 3;
    o[0] = s_abs; o[1] = s_sum; o[2] = s_sq;
  }
}

// one CTA per block: the parts are added in a fixed order (strided over the threads, then the block tree)
__global__ void __launch_bounds__(128) weight_stats_finish_kernel(const double* part, int parts, double count,
                                                                  int accumulate, double* stats) {
  __shared__ double sm[33];
  const int64_t b = blockIdx.x;
  double s[3] = {0.0, 0.0, 0.0};
  for (int p = threadIdx.x; p < parts; p += blockDim.x)
#pragma unroll
    for (int j = 0; j < 3; ++j) s[j] += part[(b * parts + p) * 3 + j];
#pragma unroll
  for (int j = 0; j < 3; ++j) s[j] = block_sum_bcast(s[j], sm);
  if (threadIdx.x == 0) {
    double* o = stats + b * 4;
    if (accumulate) { o[0] += s[0]; o[1] += s[1]; o[2] += s[2]; o[3] += count; }
    else { o[0] = s[0]; o[1] = s[1]; o[2] = s[2]; o[3] = count; }
  }
}

// One thread per layer: I_attn[l] = gamma^(l+1) rho sum_h (l1 + 0.1 var + 0.01 l2), I_mlp[l] = gamma^(l+1) sum_m
// (l1 + 0.05 var), from {sum |w|, sum w, sum w^2, count} per head / per matrix.
__global__ void distribute_importance_kernel(const double* head_stats, int n_heads, const double* fc_stats, int n_fc,
                                             int L, double rho, double gamma, double* I_attn, double* I_mlp) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= L) return;
  const double dl = pow(gamma, (double)(l + 1));
  if (head_stats && I_attn) {
    double acc = 0.0;
    for (int h = 0; h < n_heads; ++h) {
      const double* s = head_stats + ((int64_t)l * n_heads + h) * 4;
      const double c = s[3] > 0.0 ? s[3] : 1.0, mean = s[1] / c;
      acc += s[0] + 0.1 * (s[2] / c - mean * mean) + 0.01 * sqrt(s[2]);
    }
    I_attn[l] = dl * rho * acc;
  }
  if (fc_stats && I_mlp) {
    double acc = 0.0;
    for (int q = 0; q < n_fc; ++q) {
      const double* s = fc_stats + ((int64_t)l * n_fc + q) * 4;
      const double c = s[3] > 0.0 ? s[3] : 1.0, mean = s[1] / c;
      acc += s[0] + 0.05 * (s[2] / c - mean * mean);
    }
    I_mlp[l] = dl * acc;
  }
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

// Vector form of the kernel above for four tensors of one dtype with 16-byte aligned rows: a lane owns V = 16 / sizeof(T)
// adjacent columns (one 16-byte load per tensor and row), the 8 warps of a block take every 8th row of the block's
// range, two rows (8 loads) in flight per thread.  grid (column groups of 32 V, row blocks).
template <typename T>
struct L1Vec;
template <>
struct L1Vec<float> {
  static constexpr int V = 4;
  typedef float4 Raw;
  __device__ static Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ static float get(const Raw& v, int j) { return j == 0 ? v.x : j == 1 ? v.y : j == 2 ? v.z : v.w; }
};
template <>
struct L1Vec<__nv_bfloat16> {
  static constexpr int V = 8;
  typedef uint4 Raw;
  __device__ static Raw zero() { return make_uint4(0u, 0u, 0u, 0u); }
  __device__ static float get(const Raw& v, int j) {
    const uint32_t w = (j >> 1) == 0 ? v.x : (j >> 1) == 1 ? v.y : (j >> 1) == 2 ? v.z : v.w;
    return __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16));
  }
};

template <typename T>
__global__ void __launch_bounds__(256, 2) lemma1_partials_vec_kernel(const T* __restrict__ b, const T* __restrict__ c,
                                                                     const T* __restrict__ dd,
                                                                     const T* __restrict__ tt, int64_t ldb,
                                                                     int64_t ldc, int64_t ldd, int64_t ldt, int64_t N,
                                                                     int64_t cols, double* part) {
  typedef typename L1Vec<T>::Raw Raw;
  constexpr int V = L1Vec<T>::V, CB = 32 * V;
  __shared__ double red[8][CB + 1];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int row_blocks = (int)gridDim.y;
  const int64_t c0 = (int64_t)blockIdx.x * CB + (int64_t)V * lane;    // cols % V == 0: a lane is all in or all out
  const int64_t rows_per = ceil_div(N, (int64_t)row_blocks);
  const int64_t r0 = (int64_t)blockIdx.y * rows_per;
  const int64_t r1 = (r0 + rows_per < N) ? r0 + rows_per : N;
  double num[V], den[V];
#pragma unroll
  for (int j = 0; j < V; ++j) num[j] = den[j] = 0.0;
  if (c0 < cols) {
    for (int64_t rb = r0 + warp; rb < r1; rb += 16) {
      Raw raw[2][4];    // the packed loads of two rows stay in flight; values are unpacked one column at a time
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int64_t r = rb + 8 * q;
        if (r < r1) {
          raw[q][0] = *reinterpret_cast<const Raw*>(b + r * ldb + c0);
          raw[q][1] = *reinterpret_cast<const Raw*>(c + r * ldc + c0);
          raw[q][2] = *reinterpret_cast<const Raw*>(dd + r * ldd + c0);
          raw[q][3] = *reinterpret_cast<const Raw*>(tt + r * ldt + c0);
        } else {
          raw[q][0] = raw[q][1] = raw[q][2] = raw[q][3] = L1Vec<T>::zero();
        }
      }
#pragma unroll
      for (int q = 0; q < 2; ++q)
#pragma unroll
        for (int j = 0; j < V; ++j) {
          const double xb = L1Vec<T>::get(raw[q][0], j), xc = L1Vec<T>::get(raw[q][1], j);
          const double xd = L1Vec<T>::get(raw[q][2], j), xt = L1Vec<T>::get(raw[q][3], j);
          num[j] += xc * xb + xd * xt;
          den[j] += xc * xc + xd * xd;
        }
    }
  }
  // cross-warp sums in a fixed order, numerators then denominators
  for (int pass = 0; pass < 2; ++pass) {
    __syncthreads();
#pragma unroll
    for (int j = 0; j < V; ++j) red[warp][V * lane + j] = pass == 0 ? num[j] : den[j];
    __syncthreads();
    for (int cc = t; cc < CB; cc += 256) {
      const int64_t col = (int64_t)blockIdx.x * CB + cc;
      if (col < cols) {
        double sum = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) sum += red[w][cc];
        part[((int64_t)blockIdx.y * cols + col) * 2 + pass] = sum;
      }
    }
  }
}

// colred[j] = (sum over row blocks of the numerators, of the denominators) of column j
__global__ void __launch_bounds__(256) lemma1_colred_kernel(const double* __restrict__ part, int row_blocks,
                                                            int64_t cols, double* colred) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= cols) return;
  const double2* p2 = reinterpret_cast<const double2*>(part);
  double num = 0.0, den = 0.0;
  int r = 0;
  for (; r + 8 <= row_blocks; r += 8) {
    double2 v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = p2[(int64_t)(r + q) * cols + j];
#pragma unroll
    for (int q = 0; q < 8; ++q) { num += v[q].x; den += v[q].y; }
  }
  for (; r < row_blocks; ++r) {
    const double2 v = p2[(int64_t)r * cols + j];
    num += v.x;
    den += v.y;
  }
  reinterpret_cast<double2*>(colred)[j] = make_double2(num, den);
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
// One block per temperature of a grid (blockIdx.x): T = T_list[b] (T_list != nullptr) or the scalar T, multiplied by
// mean_l |I_l| when T_relative; outputs row b of r_out / k_out ([grid, L]).
__global__ void __launch_bounds__(1024) allocate_kernel(const double* I, const int64_t* n_units, int L, double rbar,
                                                        double T, const double* T_list, int T_relative, int mode,
                                                        double clip_hi, double* r_out, int64_t* k_out) {
  __shared__ double sm[33];
  const int t = threadIdx.x;
  r_out += (int64_t)blockIdx.x * L;
  k_out += (int64_t)blockIdx.x * L;
  if (T_list) T = T_list[blockIdx.x];
  if (T_relative) {
    double a = 0.0;
    for (int l = t; l < L; l += blockDim.x) a += fabs(I[l]);
    T *= block_sum_bcast(a, sm) / (double)L;
  }
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

// exclusive scan of a pair of counts over the block (1024 threads max, every thread calls it);
// returns the exclusive prefixes, the block totals through *total
__device__ int2 block_excl_scan2(int a, int b, int2* warp_tot, int2* total) {
  const int l = threadIdx.x & 31, w = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int va = __shfl_up_sync(0xffffffffu, ia, o), vb = __shfl_up_sync(0xffffffffu, ib, o);
    if (l >= o) { ia += va; ib += vb; }
  }
  __syncthreads();
  if (l == 31) warp_tot[w] = make_int2(ia, ib);
  __syncthreads();
  if (w == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    int2 v = l < nw ? warp_tot[l] : make_int2(0, 0);
    int sa = v.x, sb = v.y;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int va = __shfl_up_sync(0xffffffffu, sa, o), vb = __shfl_up_sync(0xffffffffu, sb, o);
      if (l >= o) { sa += va; sb += vb; }
    }
    warp_tot[l] = make_int2(sa - v.x, sb - v.y);          // exclusive over warps
    if (l == 31) warp_tot[32] = make_int2(sa, sb);        // totals
  }
  __syncthreads();
  const int2 base = warp_tot[w];
  *total = warp_tot[32];
  return make_int2(base.x + ia - a, base.y + ib - b);
}

// Exact top-k of one score vector per block (blockIdx.x = problem of a batch): the k largest scores are kept, among
// equal scores the lower index first (radix select on order-preserving keys, 8 bits per pass from the top).
//   scores + b * ld_scores, mask + b * ld_mask, kept_idx + b * ld_idx, tau + b;  k = k_list ? k_list[b] : k_all.
// The keys are staged once in shared memory when they fit (smem_keys != 0), else re-read from global memory.
__global__ void __launch_bounds__(1024) topk_select_kernel(const float* __restrict__ scores_all, int64_t ld_scores,
                                                           int64_t n, int64_t k_all, const int64_t* k_list,
                                                           uint8_t* mask_all, int64_t ld_mask, float* tau_all,
                                                           int32_t* kept_all, int64_t ld_idx, int smem_keys,
                                                           int skip_negative) {
  extern __shared__ uint32_t s_keys[];
  __shared__ int hist_w[32][256];     // one histogram per warp: adds collide only inside a warp
  __shared__ int hist[256];
  __shared__ int2 warp_tot[33];
  __shared__ uint32_t s_prefix;
  __shared__ int64_t s_krem;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int64_t prob = blockIdx.x;
  const float* scores = scores_all + prob * ld_scores;
  uint8_t* mask = mask_all + prob * ld_mask;
  float* tau = tau_all ? tau_all + prob : nullptr;
  int32_t* kept_idx = kept_all ? kept_all + prob * ld_idx : nullptr;
  int64_t k = k_list ? k_list[prob] : k_all;
  if (k < 0 && skip_negative) return;      // this problem keeps the mask it has
  if (k < 0) k = 0;
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
          if (score_key(scores[i]) == best) { m = scores[i] != scores[i] ? -INFINITY : scores[i]; break; }
      }
      tau[0] = m;
    }
    return;
  }
  if (smem_keys) {
    for (int64_t base = 0; base < n; base += (int64_t)blockDim.x * 4) {   // four loads in flight per thread
      float v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t i = base + (int64_t)q * blockDim.x + t;
        v[q] = i < n ? scores[i] : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int64_t i = base + (int64_t)q * blockDim.x + t;
        if (i < n) s_keys[i] = score_key(v[q]);
      }
    }
  }
  if (t == 0) { s_prefix = 0u; s_krem = k; }
  __syncthreads();
  auto key_at = [&](int64_t i) -> uint32_t { return smem_keys ? s_keys[i] : score_key(scores[i]); };
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int i = t; i < 32 * 256; i += blockDim.x) (&hist_w[0][0])[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int64_t i = t; i < n; i += blockDim.x) {
      const uint32_t key = key_at(i);
      if ((key & hi_mask) == prefix) atomicAdd(&hist_w[warp][(key >> shift) & 0xffu], 1);
    }
    __syncthreads();
    if (t < 256) {
      int sum = 0;
#pragma unroll 8
      for (int w = 0; w < 32; ++w) sum += hist_w[w][t];
      hist[t] = sum;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255 - 8 l down to 248 - 8 l: walk from the largest digit down
      int c[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c[j] = hist[255 - (8 * lane + j)]; tot += c[j]; }
      int incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const int64_t rem = s_krem, excl = incl - tot;
      __syncwarp();
      if (excl < rem && rem <= (int64_t)incl) {
        int64_t r = rem - excl;
        int bin = 255 - 8 * lane;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if ((int64_t)c[j] >= r) { bin = 255 - (8 * lane + j); break; }
          r -= c[j];
        }
        s_krem = r;   // how many to take from this bin
        s_prefix = prefix | ((uint32_t)bin << shift);
      }
    }
    __syncthreads();
  }
  const uint32_t tkey = s_prefix;
  const int64_t take_eq = s_krem;  // ties at the threshold that are kept (lowest indices first)
  // thread t owns the contiguous indices [t * per, (t + 1) * per): one scan orders the whole vector
  const int64_t per = ceil_div(n, (int64_t)blockDim.x);
  const int64_t i0 = (int64_t)t * per, i1 = (i0 + per < n) ? i0 + per : n;
  int n_eq = 0, n_gt = 0;
  for (int64_t i = i0; i < i1; ++i) {
    const uint32_t key = key_at(i);
    n_eq += key == tkey;
    n_gt += key > tkey;
  }
  int2 total;
  const int2 before = block_excl_scan2(n_eq, n_gt, warp_tot, &total);
  int64_t eq_seen = before.x, gt_seen = before.y;
  for (int64_t i = i0; i < i1; ++i) {
    const uint32_t key = key_at(i);
    const bool is_eq = key == tkey;
    const bool keep = key > tkey || (is_eq && eq_seen < take_eq);
    mask[i] = (uint8_t)keep;
    if (keep && kept_idx) kept_idx[gt_seen + (eq_seen < take_eq ? eq_seen : take_eq)] = (int32_t)i;
    if (is_eq) {
      if (eq_seen == 0 && tau) {
        const float v = scores[i];
        tau[0] = v != v ? -INFINITY : v;
      }
      ++eq_seen;
    }
    gt_seen += key > tkey;
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

// perm = the kept channels in ascending order, then the pruned ones in ascending order; count[0] = kept channels
__global__ void __launch_bounds__(1024) mask_to_perm_kernel(const uint8_t* mask, int64_t n, int32_t* perm,
                                                            int32_t* count) {
  __shared__ int warp_tot[32];
  __shared__ int s_kept;
  int kept = 0;
  for (int64_t base = 0; base < n; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    int tot;
    block_excl_scan((i < n) && mask[i] != 0, warp_tot, &tot);
    kept += tot;
  }
  if (threadIdx.x == 0) { s_kept = kept; count[0] = kept; }
  __syncthreads();
  kept = s_kept;
  int64_t before = 0;
  for (int64_t base = 0; base < n; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    const int keep = (i < n) && mask[i] != 0;
    int tot;
    const int rank = block_excl_scan(keep, warp_tot, &tot);
    if (i < n) perm[keep ? before + rank : kept + (i - before - rank)] = (int32_t)i;
    before += tot;
  }
}

// flags[0] = 1 when the k kept channels of `mask` are not exactly perm[0..k) (the support the permutation was built
// from, count_old of them); flags[1] = 1 - flags[0]
__global__ void __launch_bounds__(1024) mask_changed_kernel(const uint8_t* mask, const int32_t* perm,
                                                            const int32_t* count_old, int64_t k, int32_t* flags) {
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = (int64_t)count_old[0] != k;
  __syncthreads();
  int bad = 0;
  if (!s_bad)      // (with another count the list may not be one of this mask's size at all: it is not read)
    for (int64_t a = threadIdx.x; a < k; a += blockDim.x) bad |= mask[perm[a]] == 0;
  __syncthreads();
  if (bad) s_bad = 1;
  __syncthreads();
  if (threadIdx.x == 0) {
    flags[0] = s_bad ? 1 : 0;
    flags[1] = s_bad ? 0 : 1;
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
  int64_t rb = ceil_div(148 * 8, cb);
  if (rb > rows) rb = rows;
  if (rb < 1) rb = 1;
  return (int)rb;
}

}  // namespace

int score_row_blocks(int64_t rows, int64_t cols) { return row_blocks_for(rows, cols); }

// Launch shape of wanda_scores_kernel: column groups and row blocks (about 8 resident blocks on each of 148 SMs).
static void wanda_grid(int64_t rows, int64_t cols, int64_t* col_groups, int64_t* row_blocks) {
  const int64_t cg = ceil_div(cols, (int64_t)kWsCols);
  int64_t rb = (148 * 8) / cg;
  const int64_t rb_max = ceil_div(rows, (int64_t)kWsWarps);
  if (rb > rb_max) rb = rb_max;
  if (rb < 1) rb = 1;
  *col_groups = cg;
  *row_blocks = rb;
}

// doubles of scratch: part[row_blocks][cols], colval[cols], then the tickets (32-bit, col_groups + 1 of them)
size_t wanda_scratch_doubles(int64_t rows, int64_t cols) {
  int64_t cg, rb;
  wanda_grid(rows, cols, &cg, &rb);
  return (size_t)(rb + 1) * (size_t)cols + (size_t)(cg + 2) / 2 + 1;
}

cudaError_t wanda_scores(int kind, int group, const float* W, int64_t rows, int64_t ldw, const float* colsq,
                         int64_t colsq_stride, const double* colabs, double inv_tokens, int64_t n_units,
                         float* scores, double* importance, double* scratch, cudaStream_t stream) {
  const int64_t cols = n_units * group;
  if (cols == 0) return cudaSuccess;
  int64_t cg, rb;
  wanda_grid(rows, cols, &cg, &rb);
  const int k = kind == SP_SCORE_WANDA_L2 ? 0 : 1;
  double* part = scratch;
  double* colval = scratch + (size_t)rb * cols;
  unsigned int* tickets = reinterpret_cast<unsigned int*>(colval + cols);
  const int vec_ok = (ldw % 4 == 0) && ((reinterpret_cast<uintptr_t>(W) & 15u) == 0);
  ProfScope prof(PK_SCORES, 0.0, (double)rows * (double)cols * 4.0, stream);
  cudaError_t e = cudaMemsetAsync(tickets, 0, (size_t)(cg + 1) * sizeof(unsigned int), stream);
  if (e != cudaSuccess) return e;
  count_launch();
  wanda_scores_kernel<<<dim3((unsigned)cg, (unsigned)rb), kWsWarps * 32, 0, stream>>>(
      W, rows, cols, ldw, vec_ok, k, group, colsq, colsq_stride, colabs, inv_tokens, n_units, scores, importance, part,
      colval, tickets);
  return cudaGetLastError();
}

// parts of a block's row range so that the launch has about 148 * 8 CTAs
int weight_stats_parts(int64_t n_blocks, int64_t block_rows) {
  int64_t parts = (148 * 8) / (n_blocks > 0 ? n_blocks : 1);
  if (parts > block_rows) parts = block_rows;
  if (parts < 1) parts = 1;
  if (parts > 1024) parts = 1024;
  return (int)parts;
}

cudaError_t weight_stats(const void* W, int32_t dt, int64_t ld, int64_t rows, int64_t cols, int axis, int64_t group,
                         bool accumulate, double* stats, double* scratch, cudaStream_t stream) {
  const int64_t n_blocks = group > 0 ? (axis == 0 ? rows / group : cols / group) : 1;
  if (n_blocks <= 0 || rows <= 0 || cols <= 0) return cudaSuccess;
  const int64_t block_rows = (group > 0 && axis == 0) ? group : rows;
  const int64_t block_cols = (group > 0 && axis == 1) ? group : cols;
  const int parts = weight_stats_parts(n_blocks, block_rows);
  const size_t esz = dt == SP_BF16 ? 2 : 4;
  // 16-byte pieces need aligned rows and an aligned first column of every block
  const int64_t V = 16 / (int64_t)esz;
  const bool vec_ok = (ld % V == 0) && ((reinterpret_cast<uintptr_t>(W) & 15u) == 0) && (block_cols % V == 0) &&
                      (group == 0 || axis == 0 || group % V == 0);
  ProfScope prof(PK_SCORES, 0.0, (double)rows * (double)cols * (double)esz, stream);
  count_launch();
  const dim3 grid((unsigned)n_blocks, (unsigned)parts);
  if (dt == SP_BF16)
    weight_stats_partial_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(W), ld,
                                                                         rows, cols, axis, group, vec_ok ? 1 : 0,
                                                                         scratch);
  else
    weight_stats_partial_kernel<float><<<grid, 256, 0, stream>>>(reinterpret_cast<const float*>(W), ld, rows, cols, axis,
                                                                 group, vec_ok ? 1 : 0, scratch);
  count_launch();
  weight_stats_finish_kernel<<<(unsigned)n_blocks, 128, 0, stream>>>(
      scratch, parts, (double)block_rows * (double)block_cols, accumulate ? 1 : 0, stats);
  return cudaGetLastError();
}

cudaError_t distribute_importance(const double* head_stats, int n_heads, const double* fc_stats, int n_fc, int L,
                                  double rho, double gamma, double* I_attn, double* I_mlp, cudaStream_t stream) {
  if (L <= 0) return cudaSuccess;
  count_launch();
  distribute_importance_kernel<<<(unsigned)ceil_div((int64_t)L, (int64_t)128), 128, 0, stream>>>(
      head_stats, n_heads, fc_stats, n_fc, L, rho, gamma, I_attn, I_mlp);
  return cudaGetLastError();
}

cudaError_t lemma1_scores_stream(const sp_mat& b, const sp_mat& c, const sp_mat& dd, const sp_mat& t, int group,
                                 int64_t n_units, float* scores, double* importance, double* relaxed, double r_layer,
                                 double* scratch, cudaStream_t stream) {
  const int64_t cols = n_units * group;
  const int64_t N = b.rows;
  if (cols == 0) return cudaSuccess;
  const int rb = row_blocks_for(N, cols);
  // scratch: part[rb][cols][2], colred[cols][2] (column sums over the row blocks), unit_e[cols][2] (finish kernel)
  double* part = scratch;
  double* colred = scratch + (size_t)rb * cols * 2;
  double* unit_e = colred + (size_t)cols * 2;
  ProfScope prof(PK_SCORES, 0.0, (double)N * (double)cols * (double)(dtype_size(b.dtype) + dtype_size(c.dtype) +
                                                                    dtype_size(dd.dtype) + dtype_size(t.dtype)),
                 stream);
  const int32_t dt = b.dtype;
  const int V = dt == SP_BF16 ? 8 : 4;
  auto ok = [&](const sp_mat& m) {
    return m.dtype == dt && m.ld % V == 0 && (reinterpret_cast<uintptr_t>(m.ptr) & 15u) == 0;
  };
  const bool vec = (dt == SP_BF16 || dt == SP_F32) && cols % V == 0 && ok(b) && ok(c) && ok(dd) && ok(t);
  count_launch();
  if (vec) {
    // about 148 * 8 blocks, never more row blocks than the scratch was sized for
    const int64_t cg = ceil_div(cols, (int64_t)(32 * V));
    int64_t rbv = (148 * 8) / cg;
    if (rbv > rb) rbv = rb;
    if (rbv < 1) rbv = 1;
    const dim3 grid((unsigned)cg, (unsigned)rbv);
    if (dt == SP_BF16)
      lemma1_partials_vec_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
          reinterpret_cast<const __nv_bfloat16*>(b.ptr), reinterpret_cast<const __nv_bfloat16*>(c.ptr),
          reinterpret_cast<const __nv_bfloat16*>(dd.ptr), reinterpret_cast<const __nv_bfloat16*>(t.ptr), b.ld, c.ld,
          dd.ld, t.ld, N, cols, part);
    else
      lemma1_partials_vec_kernel<float><<<grid, 256, 0, stream>>>(
          reinterpret_cast<const float*>(b.ptr), reinterpret_cast<const float*>(c.ptr),
          reinterpret_cast<const float*>(dd.ptr), reinterpret_cast<const float*>(t.ptr), b.ld, c.ld, dd.ld, t.ld, N,
          cols, part);
    count_launch();
    lemma1_colred_kernel<<<(unsigned)ceil_div(cols, (int64_t)256), 256, 0, stream>>>(part, (int)rbv, cols, colred);
    count_launch();
    lemma1_finish_kernel<<<1, 1024, 0, stream>>>(colred, 1, cols, group, n_units, scores, importance, relaxed, r_layer,
                                                 unit_e);
    return cudaGetLastError();
  }
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
  allocate_kernel<<<1, 1024, 0, stream>>>(I, n_units, L, rbar, T, nullptr, 0, mode, clip_hi, r_out, k_out);
  return cudaGetLastError();
}

cudaError_t allocate_sparsity_grid(const double* I, const int64_t* n_units, int L, double rbar, const double* T_list,
                                   int n_T, bool T_relative, int mode, double clip_hi, double* r_out, int64_t* k_out,
                                   cudaStream_t stream) {
  ProfScope prof(PK_ALLOCATE, 0.0, (double)L * 32.0 * n_T, stream);
  count_launch();
  allocate_kernel<<<n_T, 1024, 0, stream>>>(I, n_units, L, rbar, 1.0, T_list, T_relative ? 1 : 0, mode, clip_hi, r_out,
                                            k_out);
  return cudaGetLastError();
}

cudaError_t topk_select(const float* scores, int64_t n, int64_t k, uint8_t* mask, float* tau, int32_t* kept_idx,
                        cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  return topk_select_batched(scores, n, n, 1, k, nullptr, mask, n, tau, kept_idx, n, stream);
}

cudaError_t topk_select_batched(const float* scores, int64_t ld_scores, int64_t n, int64_t batch, int64_t k_all,
                                const int64_t* k_list, uint8_t* mask, int64_t ld_mask, float* tau, int32_t* kept_idx,
                                int64_t ld_idx, cudaStream_t stream, bool skip_negative) {
  if (n == 0 || batch == 0) return cudaSuccess;
  constexpr int64_t kMaxSmemKeys = 47104;      // 184 KiB of keys beside the 33 KiB of histograms
  static PerDeviceOnce attr_once;
  const cudaError_t ea = attr_once.run([] {
    return cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(kMaxSmemKeys * sizeof(uint32_t)));
  });
  if (ea != cudaSuccess) return ea;
  const int smem_keys = n <= kMaxSmemKeys ? 1 : 0;
  ProfScope prof(PK_TOPK, 0.0, (double)batch * (double)n * 5.0, stream);
  count_launch();
  topk_select_kernel<<<(unsigned)batch, 1024, smem_keys ? (size_t)n * sizeof(uint32_t) : 0, stream>>>(
      scores, ld_scores, n, k_all, k_list, mask, ld_mask, tau, kept_idx, ld_idx, smem_keys, skip_negative ? 1 : 0);
  return cudaGetLastError();
}

__global__ void fill_i32_kernel(int32_t* x, int n, int32_t v) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) x[i] = v;
}

// ---- one threshold over L * n scores with many CTAs (Appendix B, Algorithm 3): radix select in four launches, each a
// grid-wide histogram of one key byte whose last block picks the bin; then the eq / gt counts per block, and the mask.
// state (device, ints): [0..255] histogram, [256] prefix, [257..258] remaining count (lo, hi), [259] ticket,
// [260 + b] per-block count of keys equal to the threshold key (then their exclusive prefix).
constexpr int kGselThreads = 256;
constexpr int kGselPerBlock = 8192;          // keys per block
constexpr int kGselState = 260;

__global__ void gsel_init_kernel(int32_t* st, int64_t K, int nblocks) {
  for (int i = threadIdx.x; i < kGselState + nblocks; i += blockDim.x) st[i] = 0;
  __syncthreads();
  if (threadIdx.x == 0) {
    st[257] = (int32_t)(K & 0xffffffffll);
    st[258] = (int32_t)(K >> 32);
  }
}

__global__ void __launch_bounds__(kGselThreads) gsel_hist_kernel(const float* __restrict__ scores, int64_t n_row,
                                                                 int64_t ld, int64_t total, int pass, int32_t* st) {
  __shared__ int hist[256];
  __shared__ bool last;
  const int t = threadIdx.x;
  hist[t] = 0;
  __syncthreads();
  const int shift = 24 - 8 * pass;
  const uint32_t hi_mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
  const uint32_t prefix = (uint32_t)st[256];
  const int64_t e0 = (int64_t)blockIdx.x * kGselPerBlock;
  const int64_t e1 = e0 + kGselPerBlock < total ? e0 + kGselPerBlock : total;
  for (int64_t e = e0 + t; e < e1; e += kGselThreads) {
    const uint32_t key = score_key(scores[(e / n_row) * ld + e % n_row]);
    if ((key & hi_mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xffu], 1);
  }
  __syncthreads();
  if (hist[t]) atomicAdd(&st[t], hist[t]);
  __threadfence();
  __syncthreads();
  if (t == 0) last = atomicAdd(&st[259], 1) == (int)gridDim.x - 1;
  __syncthreads();
  if (!last) return;
  __threadfence();
  // the last block: pick the bin that holds the K-th largest key among those matching the prefix
  hist[t] = __ldcg(&st[t]);
  __syncthreads();
  if (t == 0) {
    int64_t rem = ((int64_t)(uint32_t)st[257]) | ((int64_t)st[258] << 32);
    int bin = 0;
    for (int b = 255; b >= 0; --b) {
      if ((int64_t)hist[b] >= rem) { bin = b; break; }
      rem -= hist[b];
    }
    st[256] = (int32_t)(prefix | ((uint32_t)bin << shift));
    st[257] = (int32_t)(rem & 0xffffffffll);
    st[258] = (int32_t)(rem >> 32);
    st[259] = 0;
  }
  __syncthreads();
  st[t] = 0;     // histogram of the next pass
}

// per-block counts of keys equal to the threshold key; the last block turns them into exclusive prefixes
__global__ void __launch_bounds__(kGselThreads) gsel_count_kernel(const float* __restrict__ scores, int64_t n_row,
                                                                  int64_t ld, int64_t total, int32_t* st) {
  __shared__ int cnt;
  __shared__ bool last;
  const int t = threadIdx.x;
  if (t == 0) cnt = 0;
  __syncthreads();
  const uint32_t tkey = (uint32_t)st[256];
  const int64_t e0 = (int64_t)blockIdx.x * kGselPerBlock;
  const int64_t e1 = e0 + kGselPerBlock < total ? e0 + kGselPerBlock : total;
  int c = 0;
  for (int64_t e = e0 + t; e < e1; e += kGselThreads) c += score_key(scores[(e / n_row) * ld + e % n_row]) == tkey;
  if (c) atomicAdd(&cnt, c);
  __syncthreads();
  if (t == 0) {
    st[kGselState + blockIdx.x] = cnt;
    __threadfence();
    last = atomicAdd(&st[259], 1) == (int)gridDim.x - 1;
  }
  __syncthreads();
  if (!last) return;
  __threadfence();
  if (t == 0) {
    int run = 0;
    for (unsigned b = 0; b < gridDim.x; ++b) {
      const int v = __ldcg(&st[kGselState + b]);
      st[kGselState + b] = run;
      run += v;
    }
    st[259] = 0;
  }
}

// mask: keys above the threshold key are kept, equal keys in (layer, index) order until the remaining count is used up
// (a block walks its keys in order: thread t owns a contiguous run).  counts[l] += kept units of layer l.
__global__ void __launch_bounds__(kGselThreads) gsel_mask_kernel(const float* __restrict__ scores, int64_t n_row,
                                                                 int64_t ld, int64_t ld_mask, int64_t total,
                                                                 const int32_t* st, uint8_t* mask, float* tau,
                                                                 int32_t* counts) {
  __shared__ int warp_tot[32];
  const int t = threadIdx.x;
  const uint32_t tkey = (uint32_t)st[256];
  const int64_t take_eq = ((int64_t)(uint32_t)st[257]) | ((int64_t)st[258] << 32);
  const int64_t eq_before_block = st[kGselState + blockIdx.x];
  const int64_t e0 = (int64_t)blockIdx.x * kGselPerBlock;
  const int64_t e1 = e0 + kGselPerBlock < total ? e0 + kGselPerBlock : total;
  constexpr int per = kGselPerBlock / kGselThreads;
  const int64_t i0 = e0 + (int64_t)t * per, i1 = (i0 + per < e1) ? i0 + per : e1;
  int n_eq = 0;
  for (int64_t e = i0; e < i1; ++e) n_eq += score_key(scores[(e / n_row) * ld + e % n_row]) == tkey;
  // exclusive scan of n_eq over the block
  const int lane = t & 31, w = t >> 5;
  int incl = n_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[w] = incl;
  __syncthreads();
  int base = 0;
  for (int i = 0; i < w; ++i) base += warp_tot[i];
  int64_t eq_seen = eq_before_block + base + incl - n_eq;
  int kept_here = 0;
  int64_t cur_layer = i0 < i1 ? i0 / n_row : 0;
  for (int64_t e = i0; e < i1; ++e) {
    const int64_t l = e / n_row, j = e % n_row;
    if (l != cur_layer) {
      if (kept_here) atomicAdd(&counts[cur_layer], kept_here);
      kept_here = 0;
      cur_layer = l;
    }
    const float v = scores[l * ld + j];
    const uint32_t key = score_key(v);
    const bool is_eq = key == tkey;
    const bool keep = key > tkey || (is_eq && eq_seen < take_eq);
    mask[l * ld_mask + j] = (uint8_t)keep;
    kept_here += keep;
    if (is_eq) {
      if (eq_seen == 0 && tau) tau[0] = v != v ? -INFINITY : v;
      ++eq_seen;
    }
  }
  if (kept_here) atomicAdd(&counts[cur_layer], kept_here);
}

// layers left with fewer than min_keep units keep their own min_keep best: k_fix[l] = min_keep there, -1 elsewhere
__global__ void gsel_repair_list_kernel(int32_t* counts, int L, int64_t min_keep, int64_t n_row, int64_t* k_fix,
                                        int64_t* counts_out) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= L) return;
  const int64_t mk = min_keep < n_row ? min_keep : n_row;
  const bool fix = counts[l] < mk;
  k_fix[l] = fix ? mk : -1;
  counts_out[l] = fix ? mk : counts[l];
}

// counts[l] = kept units of layer l of an L x n mask (rows ld apart); one block per layer
__global__ void __launch_bounds__(256) mask_row_counts_kernel(const uint8_t* __restrict__ mask, int64_t n, int64_t ld,
                                                              int32_t* __restrict__ counts) {
  __shared__ int sm[256];
  int c = 0;
  for (int64_t j = threadIdx.x; j < n; j += 256) c += mask[(int64_t)blockIdx.x * ld + j] != 0;
  sm[threadIdx.x] = c;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) counts[blockIdx.x] = sm[0];
}

size_t global_select_scratch_bytes(int64_t total, int L) {
  const int64_t nblocks = ceil_div(total > 0 ? total : 1, (int64_t)kGselPerBlock);
  return align_up((size_t)(kGselState + nblocks) * 4, 256) + align_up((size_t)L * 4, 256) + align_up((size_t)L * 8, 256);
}

cudaError_t global_select(const float* scores, int64_t ld_scores, int64_t n, int L, int64_t K, int64_t min_keep,
                          uint8_t* mask, int64_t ld_mask, float* tau, int64_t* counts_out, void* scratch,
                          cudaStream_t stream) {
  const int64_t total = (int64_t)L * n;
  if (total == 0) return cudaSuccess;
  const int nblocks = (int)ceil_div(total, (int64_t)kGselPerBlock);
  uint8_t* sp8 = reinterpret_cast<uint8_t*>(scratch);
  int32_t* st = reinterpret_cast<int32_t*>(sp8);
  int32_t* counts = reinterpret_cast<int32_t*>(sp8 + align_up((size_t)(kGselState + nblocks) * 4, 256));
  int64_t* k_fix = reinterpret_cast<int64_t*>(reinterpret_cast<uint8_t*>(counts) + align_up((size_t)L * 4, 256));
  ProfScope prof(PK_TOPK, 0.0, (double)total * 25.0, stream);
  cudaError_t e = cudaMemsetAsync(counts, 0, (size_t)L * 4, stream);
  if (e != cudaSuccess) return e;
  constexpr int64_t kOneCtaKeys = 47104;      // what the one-CTA select keeps in shared memory
  if (K > 0 && K < total && total <= kOneCtaKeys && ld_scores == n && ld_mask == n) {
    // few keys in one contiguous array: the one-CTA select over the concatenation is faster than the launch chain
    e = topk_select(scores, total, K, mask, tau, nullptr, stream);
    if (e != cudaSuccess) return e;
    count_launch();
    mask_row_counts_kernel<<<L, 256, 0, stream>>>(mask, n, ld_mask, counts);
  } else if (K <= 0 || K >= total) {      // nothing or everything kept: no threshold to find
    e = cudaMemset2DAsync(mask, (size_t)ld_mask, K > 0 ? 1 : 0, (size_t)n, (size_t)L, stream);
    if (e != cudaSuccess) return e;
    count_launch();
    gsel_init_kernel<<<1, 256, 0, stream>>>(st, 0, nblocks);
    // counts = n or 0 per layer through the repair list below
    e = cudaMemsetAsync(counts, 0, (size_t)L * 4, stream);
    if (e != cudaSuccess) return e;
    if (K > 0) {
      count_launch();
      fill_i32_kernel<<<(L + 255) / 256, 256, 0, stream>>>(counts, L, (int32_t)n);
    }
    if (tau) {
      e = cudaMemsetAsync(tau, 0xff, sizeof(float), stream);       // NaN: no threshold
      if (e != cudaSuccess) return e;
    }
  } else {
    count_launch(7);
    gsel_init_kernel<<<1, 256, 0, stream>>>(st, K, nblocks);
    for (int pass = 0; pass < 4; ++pass)
      gsel_hist_kernel<<<nblocks, kGselThreads, 0, stream>>>(scores, n, ld_scores, total, pass, st);
    gsel_count_kernel<<<nblocks, kGselThreads, 0, stream>>>(scores, n, ld_scores, total, st);
    gsel_mask_kernel<<<nblocks, kGselThreads, 0, stream>>>(scores, n, ld_scores, ld_mask, total, st, mask, tau, counts);
  }
  count_launch();
  gsel_repair_list_kernel<<<(L + 255) / 256, 256, 0, stream>>>(counts, L, min_keep, n, k_fix, counts_out);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (min_keep > 0)   // per-layer top-k where the threshold left too few units (layers with k_fix < 0 are skipped)
    e = topk_select_batched(scores, ld_scores, n, L, 0, k_fix, mask, ld_mask, nullptr, nullptr, 0, stream, true);
  return e;
}

cudaError_t mask_to_index(const uint8_t* mask, int64_t n, int32_t* kept_idx, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  count_launch();
  mask_to_index_kernel<<<1, 1024, 0, stream>>>(mask, n, kept_idx);
  return cudaGetLastError();
}

__global__ void scale_block_kernel(float* C, int64_t ld, int64_t rows, int64_t cols, const int32_t* f_bits, int power,
                                   const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;   // conditional launch (see SkipScope)
  const float f = __int_as_float(f_bits[0]);
  const float s = power == 2 ? f * f : f;
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x)
    C[(e / cols) * ld + (e % cols)] *= s;
}

__global__ void unpermute_gram_kernel(const float* __restrict__ Gp, const int32_t* __restrict__ perm, int64_t n,
                                      float* __restrict__ G) {
  const int64_t total = n * n;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / n, j = e % n;
    // entry (i, j) of the permuted matrix from its lower triangle
    const float v = i >= j ? Gp[i * n + j] : Gp[j * n + i];
    G[(int64_t)perm[i] * n + perm[j]] = v;
  }
}

__global__ void unpermute_cols_kernel(const float* __restrict__ Rp, const int32_t* __restrict__ perm, int64_t rows,
                                      int64_t n, float* __restrict__ R) {
  const int64_t total = rows * n;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = e / n, j = e % n;
    R[r * n + perm[j]] = Rp[e];
  }
}

__global__ void decay_tag_set_kernel(int32_t* tag, int k, float c, int valid, int h_ld, int h_chunk) {
  tag[1] = valid ? k : -1;
  tag[2] = __float_as_int(c);
  tag[4] = valid ? h_ld : 0;
  tag[5] = valid ? h_chunk : 0;
}

__global__ void h_next_ready_kernel(const int32_t* same, const int32_t* tag, int h_ld, int h_chunk, int32_t* ready) {
  ready[0] = (same[0] != 0 && tag[4] == h_ld && tag[5] == h_chunk && h_ld > 0) ? 1 : 0;
  ready[1] = 1 - ready[0];
}

__global__ void unpermute_rows_kernel(const float* __restrict__ Rp, const int32_t* __restrict__ perm, int64_t n,
                                      int64_t cols, float* __restrict__ R) {
  const int64_t total = n * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    R[(int64_t)perm[i] * cols + j] = Rp[e];
  }
}

cudaError_t scale_block(float* C, int64_t ld, int64_t rows, int64_t cols, const int32_t* f_bits, int power,
                        cudaStream_t stream) {
  if (rows * cols <= 0) return cudaSuccess;
  count_launch();
  scale_block_kernel<<<(unsigned)std::min<int64_t>(ceil_div(rows * cols, (int64_t)256), 148 * 16), 256, 0, stream>>>(
      C, ld, rows, cols, f_bits, power, skip_flag());
  return cudaGetLastError();
}

cudaError_t unpermute_gram(const float* Gp, const int32_t* perm, int64_t n, float* G, cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  count_launch();
  unpermute_gram_kernel<<<(unsigned)std::min<int64_t>(ceil_div(n * n, (int64_t)256), 148 * 32), 256, 0, stream>>>(Gp, perm,
                                                                                                               n, G);
  return cudaGetLastError();
}

cudaError_t unpermute_cols(const float* Rp, const int32_t* perm, int64_t rows, int64_t n, float* R,
                           cudaStream_t stream) {
  if (rows * n <= 0) return cudaSuccess;
  count_launch();
  unpermute_cols_kernel<<<(unsigned)std::min<int64_t>(ceil_div(rows * n, (int64_t)256), 148 * 32), 256, 0, stream>>>(
      Rp, perm, rows, n, R);
  return cudaGetLastError();
}

cudaError_t decay_tag_set(int32_t* tag, int64_t k, float c, bool valid, int64_t h_ld, int64_t h_chunk,
                          cudaStream_t stream) {
  count_launch();
  decay_tag_set_kernel<<<1, 1, 0, stream>>>(tag, (int)k, c, valid ? 1 : 0, (int)h_ld, (int)h_chunk);
  return cudaGetLastError();
}

cudaError_t h_next_ready(const int32_t* same, const int32_t* tag, int64_t h_ld, int64_t h_chunk, int32_t* ready,
                         cudaStream_t stream) {
  count_launch();
  h_next_ready_kernel<<<1, 1, 0, stream>>>(same, tag, (int)h_ld, (int)h_chunk, ready);
  return cudaGetLastError();
}

cudaError_t unpermute_rows(const float* Rp, const int32_t* perm, int64_t n, int64_t cols, float* R,
                           cudaStream_t stream) {
  if (n * cols <= 0) return cudaSuccess;
  count_launch();
  unpermute_rows_kernel<<<(unsigned)std::min<int64_t>(ceil_div(n * cols, (int64_t)256), 148 * 32), 256, 0, stream>>>(
      Rp, perm, n, cols, R);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(1024) mask_count_check_kernel(const uint8_t* mask, int64_t n, int64_t k,
                                                                int32_t* status) {
  __shared__ int warp_tot[32];
  int kept = 0;
  for (int64_t base = 0; base < n; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    int tot;
    block_excl_scan((i < n) && mask[i] != 0, warp_tot, &tot);
    kept += tot;
  }
  if (threadIdx.x == 0 && kept != k) report_status(status, SP_ERR_SHAPE, kept, 21);
}

cudaError_t mask_count_check(const uint8_t* mask, int64_t n, int64_t k, int32_t* status, cudaStream_t stream) {
  if (status == nullptr) return cudaSuccess;
  count_launch();
  mask_count_check_kernel<<<1, 1024, 0, stream>>>(mask, n, k, status);
  return cudaGetLastError();
}

cudaError_t mask_to_perm(const uint8_t* mask, int64_t n, int32_t* perm, int32_t* count, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  count_launch();
  mask_to_perm_kernel<<<1, 1024, 0, stream>>>(mask, n, perm, count);
  return cudaGetLastError();
}

cudaError_t mask_changed(const uint8_t* mask, const int32_t* perm, const int32_t* count_old, int64_t k, int32_t* flags,
                         cudaStream_t stream) {
  count_launch();
  mask_changed_kernel<<<1, 1024, 0, stream>>>(mask, perm, count_old, k, flags);
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
  // the partial sums take (row_blocks + 1) x cols doubles; row_blocks shrinks as cols grows, so the product stays
  // bounded
  if (sp::wanda_scratch_doubles(in->W.rows, cols) > kStaticScratchDoubles) return SP_ERR_STATIC_LIMIT;
  double* scratch = nullptr;
  const sp_status st = static_scratch_address(&scratch);
  if (st != SP_OK) return st;
  // every partial sum that is read was written earlier in this same call, so nothing an earlier call left behind
  // is read; only the few arrival tickets are cleared (a memset on the stream, no allocation)
  if (sp::wanda_scores(kind, group, reinterpret_cast<const float*>(in->W.ptr), in->W.rows, in->W.ld, in->colsq,
                       in->colsq_stride, in->colabs, in->inv_tokens, n_units, scores, layer_importance, scratch,
                       reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SP_ERR_CUDA;
  return SP_OK;
}
