// fp32 Cholesky factorisation and triangular solves whose O(n^3) / O(m n^2) work runs on the tensor cores.
//
// The regularised weight recovery W = R (G + rho I)^-1 needs fp32-level accuracy (G is a Gram matrix of ReLU
// activations with a condition number of the order of its size), which a plain bf16 product cannot give.  Every fp32
// value is therefore held as an exact sum of three bf16 parts (hi + mid + lo, 3 x 8 mantissa bits), and a product
// of two such operands is taken as the six part products of weight >= 2^-16 (hi.hi, hi.mid, mid.hi, hi.lo, lo.hi,
// mid.mid), each a K segment of one tcgen05 GEMM with fp32 accumulation.  The dropped terms are below 2^-23.
//
// Blocked right-looking algorithm with 128-wide panels:
//   diagonal block : one CTA factorises it in registers (4 x 4 elements per thread) and forms inv(L11) in the same
//                    sweep (the row operations of the elimination applied to an identity block);
//   panel          : L21 = A21 inv(L11)^T on the CUDA cores (K = 128), written as fp32 and as the three bf16 parts;
//   trailing update: A22 -= L21 L21^T (lower triangle) as one six-segment tensor-core GEMM.
// The triangular solves X L^T = R, W L = X use the same two kernels block column by block column.
#include "sp_common.cuh"

namespace sp {
namespace {

constexpr int TB = kCholTcNB;          // 128
constexpr int DIAG_BLOCKS = (TB / 4) * (TB / 4 + 1) / 2;   // 528 lower-triangular 4 x 4 blocks
constexpr int DIAG_THREADS = 544;      // 17 warps

// Factorise the nb x nb diagonal block at A (lower triangle) and write L back; dinv (TB x TB, row-major) receives
// inv(L), zero above the diagonal, identity on the padding rows nb..TB-1.  A non-positive pivot is reported once
// through `status` and replaced by 1.
//
// Elimination without square roots in the loop: step j subtracts a_ij a_cj / p_j from the trailing part (p_j the
// pivot), and applies the same row operations to an identity block B.  At the end L_ic = a_ic / sqrt(p_c) and
// inv(L)_ic = B_ic / sqrt(p_i).
__global__ void __launch_bounds__(DIAG_THREADS) chol_diag128_kernel(float* A, int64_t lda, int nb, float* dinv,
                                                                    int64_t row0, int32_t* status) {
  __shared__ float colbuf[2][TB];   // column j of the trailing matrix (unscaled), double buffered
  __shared__ float rowbuf[2][TB];   // row j of B
  __shared__ float piv[TB];
  const int t = threadIdx.x;
  const bool active = t < DIAG_BLOCKS;
  // t = bi (bi + 1) / 2 + bj with bj <= bi
  int bi = (int)((sqrtf(8.f * (float)t + 1.f) - 1.f) * 0.5f);
  while ((bi + 1) * (bi + 2) / 2 <= t) ++bi;
  while (bi * (bi + 1) / 2 > t) --bi;
  const int bj = t - bi * (bi + 1) / 2;

  float a[4][4], b[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int i = 4 * bi + r, c = 4 * bj + s;
      float v = 0.f;
      if (active && i < nb && c <= i) v = A[(int64_t)i * lda + c];
      if (i >= nb && i == c) v = 1.f;
      a[r][s] = v;
      b[r][s] = (i == c) ? 1.f : 0.f;
    }
  if (t < TB) piv[t] = 1.f;
  // zero the part of dinv that no thread owns (blocks strictly above the diagonal)
  for (int e = t; e < TB * TB; e += DIAG_THREADS) {
    const int i = e / TB, c = e % TB;
    if ((c >> 2) > (i >> 2)) dinv[e] = 0.f;
  }
  __syncthreads();

  for (int jb = 0; jb < TB / 4; ++jb) {
    if (jb * 4 >= nb) break;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = jb * 4 + jj;
      if (j < nb) {                     // uniform over the block
        const int buf = j & 1;
        if (active && bj == jb) {       // owners of column j
#pragma unroll
          for (int r = 0; r < 4; ++r) colbuf[buf][4 * bi + r] = a[r][jj];
          if (bi == jb) {
            float p = a[jj][jj];
            if (!(p > 0.f)) {
              report_status(status, SP_ERR_NOT_SPD, (int32_t)(row0 + j), 0);
              p = 1.f;
              a[jj][jj] = 1.f;
              colbuf[buf][j] = 1.f;
            }
            piv[j] = p;
          }
        }
        if (active && bi == jb) {       // owners of row j of B
#pragma unroll
          for (int s = 0; s < 4; ++s) rowbuf[buf][4 * bj + s] = b[jj][s];
        }
        __syncthreads();
        if (active && 4 * bi + 3 > j) {
          const float inv = 1.f / colbuf[buf][j];
          float cr[4], cc[4], rb[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) cr[r] = colbuf[buf][4 * bi + r] * inv;
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            cc[s] = colbuf[buf][4 * bj + s];
            rb[s] = rowbuf[buf][4 * bj + s];
          }
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              const int i = 4 * bi + r, c = 4 * bj + s;
              if (i > j) {
                if (c > j) a[r][s] -= cr[r] * cc[s];
                else b[r][s] -= cr[r] * rb[s];
              }
            }
        }
      }
    }
  }
  __syncthreads();
  if (active) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = 4 * bi + r;
      const float inv_sqrt_i = rsqrtf(piv[i]);
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int c = 4 * bj + s;
        if (c <= i) {
          if (i < nb) A[(int64_t)i * lda + c] = a[r][s] / sqrtf(piv[c]);
          dinv[i * TB + c] = b[r][s] * inv_sqrt_i;
        } else {
          dinv[i * TB + c] = 0.f;
        }
      }
    }
  }
}

__device__ __forceinline__ void split3(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(hi);
  mid = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(mid);
  lo = __float2bfloat16_rn(r2);
}

constexpr int PA_ROWS = 64;
constexpr int PA_THREADS = 256;
constexpr size_t PA_SMEM = (size_t)(TB + PA_ROWS) * (TB + 1) * sizeof(float);

// X[i, 0:nb] <- X[i, 0:nb] inv(L)^T (TRANS == false) or X[i, 0:nb] inv(L) (TRANS == true), for `rows` rows.
// dinv is the TB x TB block written by chol_diag128_kernel.  The result is written back in fp32 (write_f32) and as
// three bf16 parts to S[i * lds + part * s_seg + c] for all TB columns (zero beyond nb).
template <bool TRANS>
__global__ void __launch_bounds__(PA_THREADS) panel_apply_kernel(float* X, int64_t ldx, int64_t rows, int nb,
                                                                 const float* __restrict__ dinv, __nv_bfloat16* S,
                                                                 int64_t lds, int64_t s_seg, int write_f32) {
  extern __shared__ float pa_smem[];
  float (*Lt)[TB + 1] = reinterpret_cast<float (*)[TB + 1]>(pa_smem);               // Lt[k][c]
  float (*As)[TB + 1] = reinterpret_cast<float (*)[TB + 1]>(pa_smem + TB * (TB + 1));  // As[row][k]
  const int t = threadIdx.x;
  const int64_t r0 = (int64_t)blockIdx.x * PA_ROWS;
  for (int e = t; e < TB * TB; e += PA_THREADS) {
    const int u = e / TB, v = e % TB;          // dinv[u][v], v contiguous
    if (TRANS) Lt[u][v] = dinv[e];             // Lt[k][c] = inv(L)[k][c]
    else Lt[v][u] = dinv[e];                   // Lt[k][c] = inv(L)[c][k]
  }
  for (int e = t; e < PA_ROWS * TB; e += PA_THREADS) {
    const int i = e / TB, k = e % TB;
    const int64_t gi = r0 + i;
    As[i][k] = (gi < rows && k < nb) ? X[gi * ldx + k] : 0.f;
  }
  __syncthreads();
  const int tx = t & 15, ty = t >> 4;          // 16 column groups (columns tx + 16 j), 16 row groups of 4 rows
  float acc[4][8];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[r][j] = 0.f;
#pragma unroll 4
  for (int k = 0; k < TB; ++k) {
    float av[4], lv[8];
#pragma unroll
    for (int r = 0; r < 4; ++r) av[r] = As[ty * 4 + r][k];
#pragma unroll
    for (int j = 0; j < 8; ++j) lv[j] = Lt[k][tx + 16 * j];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int64_t gi = r0 + ty * 4 + r;
    if (gi >= rows) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = tx + 16 * j;
      const float v = (c < nb) ? acc[r][j] : 0.f;
      if (write_f32 && c < nb) X[gi * ldx + c] = v;
      if (S) {
        __nv_bfloat16 hi, mid, lo;
        split3(v, hi, mid, lo);
        __nv_bfloat16* dst = S + gi * lds + c;
        dst[0] = hi;
        dst[s_seg] = mid;
        dst[2 * s_seg] = lo;
      }
    }
  }
}

template <bool TRANS>
cudaError_t launch_panel_apply(float* X, int64_t ldx, int64_t rows, int nb, const float* dinv, __nv_bfloat16* S,
                               int64_t lds, int64_t s_seg, bool write_f32, cudaStream_t stream) {
  static bool attr = false;
  if (!attr) {
    cudaError_t e = cudaFuncSetAttribute(panel_apply_kernel<TRANS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)PA_SMEM);
    if (e != cudaSuccess) return e;
    attr = true;
  }
  if (rows <= 0) return cudaSuccess;
  count_launch();
  panel_apply_kernel<TRANS><<<(unsigned)ceil_div(rows, PA_ROWS), PA_THREADS, PA_SMEM, stream>>>(
      X, ldx, rows, nb, dinv, S, lds, s_seg, write_f32 ? 1 : 0);
  return cudaGetLastError();
}

// The six kept part products of two three-part operands: A parts (hi, hi, mid, hi, lo, mid) against B parts
// (hi, mid, hi, lo, hi, mid).
constexpr int kPartA[6] = {0, 0, 1, 0, 2, 1};
constexpr int kPartB[6] = {0, 1, 0, 2, 0, 1};

}  // namespace

int64_t chol_tc_pad(int64_t n) { return (n + TB - 1) / TB * TB; }

sp_status potrf_lower_tc(float* A, int64_t n, int64_t lda, float* dinv, void* Pv, int32_t* status_dev,
                         cudaStream_t stream) {
  __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(Pv);
  const int64_t np = chol_tc_pad(n), ldp = 3 * np;
  for (int64_t k0 = 0; k0 < n; k0 += TB) {
    const int nb = (int)((n - k0 < TB) ? (n - k0) : TB);
    float* dk = dinv + (k0 / TB) * TB * TB;
    count_launch();
    chol_diag128_kernel<<<1, DIAG_THREADS, 0, stream>>>(A + k0 * lda + k0, lda, nb, dk, k0, status_dev);
    if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    const int64_t rem = n - k0 - nb;
    if (rem <= 0) break;
    // L21 = A21 inv(L11)^T, fp32 in place and as bf16 parts in P[k0+nb.., part * np + k0 ..]
    if (launch_panel_apply<false>(A + (k0 + nb) * lda + k0, lda, rem, nb, dk, P + (k0 + nb) * ldp + k0, ldp, np, true,
                                  stream) != cudaSuccess)
      return SP_ERR_CUDA;
    // A22 -= L21 L21^T on the lower triangle
    TcOperand ta{P + (k0 + nb) * ldp, ldp, true};
    ta.kext = ldp;
    ta.mnext = rem;
    TcSegments sg;
    sg.nseg = 6;
    for (int s = 0; s < 6; ++s) {
      sg.a_k[s] = (int32_t)(kPartA[s] * np + k0);
      sg.b_k[s] = (int32_t)(kPartB[s] * np + k0);
    }
    float* A22 = A + (k0 + nb) * lda + (k0 + nb);
    sp_status st = gemm_tc(rem, rem, TB, -1.f, ta, ta, 1.f, Operand{A22, SP_F32, lda, 1}, OutOperand{A22, SP_F32, lda},
                           true, status_dev, stream, &sg, (double)rem * (double)rem * (double)nb);
    if (st != SP_OK) return st;
  }
  return SP_OK;
}

sp_status potrs_right_tc(float* X, int64_t m, int64_t n, int64_t ldx, const void* Pv, const float* dinv, void* Xsv,
                         int32_t* status_dev, cudaStream_t stream) {
  const __nv_bfloat16* P = reinterpret_cast<const __nv_bfloat16*>(Pv);
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(Xsv);
  const int64_t np = chol_tc_pad(n), ldp = 3 * np;
  const int64_t lds = 3 * TB;
  TcOperand ta{Xs, lds, true};
  ta.kext = lds;
  ta.mnext = m;
  // Y L^T = X, block columns left to right
  for (int64_t j0 = 0; j0 < n; j0 += TB) {
    const int nb = (int)((n - j0 < TB) ? (n - j0) : TB);
    const float* dj = dinv + (j0 / TB) * TB * TB;
    if (launch_panel_apply<false>(X + j0, ldx, m, nb, dj, Xs, lds, TB, true, stream) != cudaSuccess) return SP_ERR_CUDA;
    const int64_t rem = n - j0 - nb;
    if (rem <= 0) break;
    // X[:, j1:] -= Y_j L[j1:, j0:j0+nb]^T : B(k, c) = L[j1 + c, j0 + k], K-major rows of P
    TcOperand tb{P + (j0 + nb) * ldp, ldp, true};
    tb.kext = ldp;
    tb.mnext = rem;
    TcSegments sg;
    sg.nseg = 6;
    for (int s = 0; s < 6; ++s) {
      sg.a_k[s] = kPartA[s] * TB;
      sg.b_k[s] = (int32_t)(kPartB[s] * np + j0);
    }
    float* Xr = X + j0 + nb;
    sp_status st = gemm_tc(m, rem, TB, -1.f, ta, tb, 1.f, Operand{Xr, SP_F32, ldx, 1}, OutOperand{Xr, SP_F32, ldx},
                           false, status_dev, stream, &sg, 2.0 * (double)m * (double)rem * (double)nb);
    if (st != SP_OK) return st;
  }
  // W L = Y, block columns right to left
  const int64_t nblk = ceil_div(n, (int64_t)TB);
  for (int64_t jb = nblk - 1; jb >= 0; --jb) {
    const int64_t j0 = jb * TB;
    const int nb = (int)((n - j0 < TB) ? (n - j0) : TB);
    const float* dj = dinv + jb * TB * TB;
    if (launch_panel_apply<true>(X + j0, ldx, m, nb, dj, Xs, lds, TB, true, stream) != cudaSuccess) return SP_ERR_CUDA;
    if (j0 == 0) break;
    // X[:, :j0] -= W_j L[j0:j0+nb, :j0] : B(k, c) = L[j0 + k, c], rows of P with the columns (N) contiguous
    TcOperand tb{P + j0 * ldp, ldp, false};
    tb.kext = n - j0;      // rows of L that exist; beyond them the tensor map returns zero
    tb.mnext = ldp;
    TcSegments sg;
    sg.nseg = 6;
    for (int s = 0; s < 6; ++s) {
      sg.a_k[s] = kPartA[s] * TB;
      sg.b_mn[s] = (int32_t)(kPartB[s] * np);
    }
    sp_status st = gemm_tc(m, j0, TB, -1.f, ta, tb, 1.f, Operand{X, SP_F32, ldx, 1}, OutOperand{X, SP_F32, ldx}, false,
                           status_dev, stream, &sg, 2.0 * (double)m * (double)j0 * (double)nb);
    if (st != SP_OK) return st;
  }
  return SP_OK;
}

}  // namespace sp
