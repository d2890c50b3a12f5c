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

// Factorise the nb x nb diagonal block at A (lower triangle), write L back, and write inv(L) and its transpose to
// dinv[0 : TB*TB] and dinv[TB*TB : 2*TB*TB] (row-major TB x TB, zero above / below the diagonal respectively,
// identity on the padding rows nb..TB-1).  A non-positive pivot is reported once through `status` and replaced by 1.
//
// One thread owns one 4 x 4 block of the lower triangle in registers.  Elimination without square roots in the
// loop: step j subtracts a_ij a_cj / p_j from the trailing columns c > j (p_j the pivot) and applies the same row
// operations to an identity block B on the columns c <= j.  A column of the trailing matrix is final when its step
// comes: it is scaled by 1/sqrt(p_j) and stored as column j of L, and its registers then carry column j of B.  So a
// single register block m holds "a" on the columns still to be eliminated and "B" on the others, and one shared
// vector w per step feeds both updates: w[i] = a_ij for i > j, w[c] = B_jc for c < j, w[j] = 1 / p_j.
// A thread owns part of the eliminated column only while j runs through its own block column, so it keeps those
// four unscaled columns in a second register block and scales them after the loop: L_ic = a_ic / sqrt(p_c),
// inv(L)_ic = B_ic / sqrt(p_i).  The loop's critical path per step is barrier, one shared load, one multiply-add.
__global__ void __launch_bounds__(DIAG_THREADS) chol_diag128_kernel(float* A, int64_t lda, int nb, float* dinv,
                                                                    int64_t row0, int32_t* status) {
  __shared__ __align__(16) float wbuf[2][TB];   // double buffered: one barrier per step
  __shared__ float piv[TB];
  const int t = threadIdx.x;
  const bool active = t < DIAG_BLOCKS;
  // t = bi (bi + 1) / 2 + bj with bj <= bi
  int bi = (int)((sqrtf(8.f * (float)t + 1.f) - 1.f) * 0.5f);
  while ((bi + 1) * (bi + 2) / 2 <= t) ++bi;
  while (bi * (bi + 1) / 2 > t) --bi;
  const int bj = t - bi * (bi + 1) / 2;

  float m[4][4], lcol[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int i = 4 * bi + r, c = 4 * bj + s;
      float v = 0.f;
      if (active && i < nb && c <= i) v = A[(int64_t)i * lda + c];
      if (i >= nb && i == c) v = 1.f;
      m[r][s] = v;
      lcol[r][s] = v;
    }
  if (t < TB) piv[t] = 1.f;
  // zero the parts of the two inverse blocks that no thread owns (blocks strictly above the diagonal of inv(L))
  for (int e = t; e < TB * TB; e += DIAG_THREADS) {
    const int i = e / TB, c = e % TB;
    if ((c >> 2) > (i >> 2)) {
      dinv[e] = 0.f;
      dinv[TB * TB + c * TB + i] = 0.f;
    }
  }
  __syncthreads();

  for (int jb = 0; jb < TB / 4; ++jb) {
    if (jb * 4 >= nb) break;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = jb * 4 + jj;
      if (j < nb) {                     // uniform over the block
        float* wb = wbuf[j & 1];
        if (active && bj == jb) {       // owners of column j: live values below the diagonal, and the pivot
#pragma unroll
          for (int r = 0; r < 4; ++r)
            if (4 * bi + r > j) wb[4 * bi + r] = m[r][jj];
          if (bi == jb) {
            float p = m[jj][jj];
            if (!(p > 0.f)) {
              report_status(status, SP_ERR_NOT_SPD, (int32_t)(row0 + j), 0);
              p = 1.f;
              m[jj][jj] = 1.f;
            }
            // reciprocal of the pivot: hardware approximation refined by one Newton step (error below 1 ulp)
            float ip;
            asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(ip) : "f"(p));
            ip = fmaf(ip, fmaf(-p, ip, 1.f), ip);
            wb[j] = ip;
            piv[j] = p;
          }
        }
        if (active && bi == jb) {       // owners of row j of B (columns left of j)
#pragma unroll
          for (int s = 0; s < 4; ++s)
            if (4 * bj + s < j) wb[4 * bj + s] = m[jj][s];
        }
        __syncthreads();
        if (active && 4 * bi + 3 >= j) {
          const float inv = wb[j];
          if (bj == jb) {               // column j is final: keep it for L, its registers now carry column j of B
#pragma unroll
            for (int r = 0; r < 4; ++r) {
              const int i = 4 * bi + r;
              if (i >= j) {
                lcol[r][jj] = m[r][jj];
                m[r][jj] = (i == j) ? 1.f : 0.f;
              }
            }
          }
          const float4 wr = *reinterpret_cast<const float4*>(&wb[4 * bi]);
          const float4 wc = *reinterpret_cast<const float4*>(&wb[4 * bj]);
          const float wrv[4] = {wr.x, wr.y, wr.z, wr.w}, wcv[4] = {wc.x, wc.y, wc.z, wc.w};
          float cr[4], w[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) cr[r] = (4 * bi + r > j) ? wrv[r] * inv : 0.f;
#pragma unroll
          for (int s = 0; s < 4; ++s) w[s] = (4 * bj + s == j) ? 1.f : wcv[s];
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int s = 0; s < 4; ++s) m[r][s] = fmaf(-cr[r], w[s], m[r][s]);
        }
      }
    }
  }
  __syncthreads();
  if (active) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = 4 * bi + r;
      const float inv_sqrt_i = 1.f / sqrtf(piv[i]);
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int c = 4 * bj + s;
        const float v = (c <= i) ? m[r][s] * inv_sqrt_i : 0.f;
        dinv[i * TB + c] = v;
        dinv[TB * TB + c * TB + i] = v;
        if (c <= i && i < nb) A[(int64_t)i * lda + c] = lcol[r][s] / sqrtf(piv[c]);
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

constexpr int PA_ROWS = 32;
constexpr int PA_THREADS = 128;
constexpr int PA_APAD = PA_ROWS + 4;
constexpr size_t PA_SMEM = ((size_t)TB * TB + (size_t)TB * PA_APAD) * sizeof(float);

// X[i, 0:nb] <- X[i, 0:nb] inv(L)^T (TRANS == false) or X[i, 0:nb] inv(L) (TRANS == true), for `rows` rows.
// dinv is the pair of TB x TB blocks written by chol_diag128_kernel.  The result is written back in fp32 (write_f32)
// and as three bf16 parts to S[i * lds + part * s_seg + c] for all TB columns (zero beyond nb).
// One CTA takes 32 rows; a thread computes 4 rows x 8 columns.
template <bool TRANS>
__global__ void __launch_bounds__(PA_THREADS) panel_apply_kernel(float* X, int64_t ldx, int64_t rows, int nb,
                                                                 const float* __restrict__ dinv, __nv_bfloat16* S,
                                                                 int64_t lds, int64_t s_seg, int write_f32) {
  extern __shared__ __align__(16) float pa_smem[];
  float (*Lt)[TB] = reinterpret_cast<float (*)[TB]>(pa_smem);                       // Lt[k][c]
  float (*At)[PA_APAD] = reinterpret_cast<float (*)[PA_APAD]>(pa_smem + TB * TB);   // At[k][row]
  const int t = threadIdx.x;
  const int64_t r0 = (int64_t)blockIdx.x * PA_ROWS;
  const bool x_al = (ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0);
  {
    // the rows of X first (the loads of all 8 float4 of a thread are in flight together) ...
    float4 xv[PA_ROWS * TB / 4 / PA_THREADS];
#pragma unroll
    for (int q = 0; q < PA_ROWS * TB / 4 / PA_THREADS; ++q) {
      const int e = t + q * PA_THREADS;
      const int i = e / (TB / 4), k = (e % (TB / 4)) * 4;
      const int64_t gi = r0 + i;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (gi < rows) {
        const float* src = X + gi * ldx + k;
        if (x_al && k + 4 <= nb) {
          v = *reinterpret_cast<const float4*>(src);
        } else {
          if (k < nb) v.x = src[0];
          if (k + 1 < nb) v.y = src[1];
          if (k + 2 < nb) v.z = src[2];
          if (k + 3 < nb) v.w = src[3];
        }
      }
      xv[q] = v;
    }
    // ... then Lt[k][c] = inv(L)[c][k] (the transposed copy) or inv(L)[k][c]: a straight copy either way
    const float4* src = reinterpret_cast<const float4*>(dinv + (TRANS ? 0 : TB * TB));
    float4* dst = reinterpret_cast<float4*>(pa_smem);
#pragma unroll 16
    for (int e = t; e < TB * TB / 4; e += PA_THREADS) dst[e] = src[e];
#pragma unroll
    for (int q = 0; q < PA_ROWS * TB / 4 / PA_THREADS; ++q) {
      const int e = t + q * PA_THREADS;
      const int i = e / (TB / 4), k = (e % (TB / 4)) * 4;
      At[k][i] = xv[q].x; At[k + 1][i] = xv[q].y; At[k + 2][i] = xv[q].z; At[k + 3][i] = xv[q].w;
    }
  }
  __syncthreads();
  const int tx = t & 15, ty = t >> 4;          // columns 8 tx .. 8 tx + 7, rows 4 ty .. 4 ty + 3
  float acc[4][8];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[r][j] = 0.f;
#pragma unroll 4
  for (int k = 0; k < TB; ++k) {
    const float4 a0 = *reinterpret_cast<const float4*>(&At[k][4 * ty]);
    const float4 l0 = *reinterpret_cast<const float4*>(&Lt[k][8 * tx]);
    const float4 l1 = *reinterpret_cast<const float4*>(&Lt[k][8 * tx + 4]);
    const float av[4] = {a0.x, a0.y, a0.z, a0.w};
    const float lv[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
  }
  const int c0 = 8 * tx;
  const bool x_vec = write_f32 && c0 + 8 <= nb && x_al;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int64_t gi = r0 + 4 * ty + r;
    if (gi >= rows) continue;
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (c0 + j < nb) ? acc[r][j] : 0.f;
    if (write_f32) {
      float* dst = X + gi * ldx + c0;
      if (x_vec) {
        *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c0 + j < nb) dst[j] = v[j];
      }
    }
    if (S) {   // S + gi * lds + part * s_seg + c0 is 16-byte aligned by construction (lds, s_seg multiples of 8)
      __align__(16) __nv_bfloat16 part[3][8];
#pragma unroll
      for (int j = 0; j < 8; ++j) split3(v[j], part[0][j], part[1][j], part[2][j]);
#pragma unroll
      for (int q = 0; q < 3; ++q)
        *reinterpret_cast<uint4*>(S + gi * lds + q * s_seg + c0) = *reinterpret_cast<const uint4*>(part[q]);
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
  ProfScope prof(PK_PANEL_APPLY, 2.0 * (double)rows * TB * TB, 0.0, stream);
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
    float* dk = dinv + (k0 / TB) * 2 * TB * TB;
    {
      count_launch();
      ProfScope prof(PK_CHOL_DIAG, (double)nb * nb * nb * (2.0 / 3.0), 0.0, stream);
      chol_diag128_kernel<<<1, DIAG_THREADS, 0, stream>>>(A + k0 * lda + k0, lda, nb, dk, k0, status_dev);
      if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    }
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
    const float* dj = dinv + (j0 / TB) * 2 * TB * TB;
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
    const float* dj = dinv + jb * 2 * TB * TB;
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
