// Blocked lower Cholesky and right-hand triangular solves for the regularised weight recovery
// W = R (G + rho I)^-1.  The O(n^3) and O(m n^2) work is expressed as GEMMs on the diagonal-block inverses;
// only the NB x NB diagonal factorisation runs in a single thread block.
#include "sp_common.cuh"

namespace sp {
namespace {

constexpr int NB = kCholNB;

template <typename T> struct DT;
template <> struct DT<float> { static constexpr int32_t v = SP_F32; };
template <> struct DT<double> { static constexpr int32_t v = SP_F64; };

// Factor the nb x nb diagonal block at A (lower), write L back, and write inv(L) (lower, zero padded to NB x NB,
// unit diagonal on the padding) to dinv.  A non-positive pivot is reported once and replaced by 1.
template <typename T>
__global__ void __launch_bounds__(256) chol_diag_kernel(T* A, int64_t lda, int nb, T* dinv, int64_t block_row0,
                                                        int32_t* status) {
  extern __shared__ __align__(16) unsigned char chol_smem[];
  T (*L)[NB + 1] = reinterpret_cast<T (*)[NB + 1]>(chol_smem);
  T (*Li)[NB + 1] = reinterpret_cast<T (*)[NB + 1]>(chol_smem + sizeof(T) * NB * (NB + 1));
  const int t = threadIdx.x;
  for (int e = t; e < NB * NB; e += blockDim.x) {
    const int i = e / NB, j = e % NB;
    T v = (T)0;
    if (i < nb && j < nb && j <= i) v = A[(int64_t)i * lda + j];
    if (i >= nb && i == j) v = (T)1;
    L[i][j] = v;
  }
  __syncthreads();
  for (int j = 0; j < nb; ++j) {
    if (t == 0) {
      T p = L[j][j];
      if (!(p > (T)0)) {
        report_status(status, SP_ERR_NOT_SPD, (int32_t)(block_row0 + j), 0);
        p = (T)1;
      }
      L[j][j] = sqrt(p);
    }
    __syncthreads();
    const T piv = L[j][j];
    for (int i = j + 1 + t; i < nb; i += blockDim.x) L[i][j] /= piv;
    __syncthreads();
    // trailing update of the lower triangle: L[i][c] -= L[i][j] * L[c][j], j < c <= i < nb
    const int rem = nb - j - 1;
    for (int e = t; e < rem * rem; e += blockDim.x) {
      const int i = j + 1 + e / rem, c = j + 1 + e % rem;
      if (c <= i) L[i][c] -= L[i][j] * L[c][j];
    }
    __syncthreads();
  }
  // inverse of the lower-triangular factor, one column per thread
  for (int c = t; c < NB; c += blockDim.x) {
    for (int i = 0; i < NB; ++i) {
      if (i < c) { Li[i][c] = (T)0; continue; }
      T s = (i == c) ? (T)1 : (T)0;
      for (int k = c; k < i; ++k) s -= L[i][k] * Li[k][c];
      Li[i][c] = s / L[i][i];
    }
  }
  __syncthreads();
  for (int e = t; e < NB * NB; e += blockDim.x) {
    const int i = e / NB, j = e % NB;
    dinv[e] = Li[i][j];
    if (i < nb && j < nb && j <= i) A[(int64_t)i * lda + j] = L[i][j];
  }
}

template <typename T>
constexpr size_t diag_smem_bytes() { return 2 * sizeof(T) * NB * (NB + 1); }

template <typename T>
cudaError_t prepare_diag_kernel() {
  static PerDeviceOnce once;           // one per instantiation; the attribute belongs to the device's context
  return once.run([] {
    return cudaFuncSetAttribute(chol_diag_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)diag_smem_bytes<T>());
  });
}

template <typename T>
inline Operand op(const T* p, int64_t s0, int64_t s1) { return Operand{p, DT<T>::v, s0, s1}; }
template <typename T>
inline OutOperand out(T* p, int64_t ld) { return OutOperand{p, DT<T>::v, ld}; }

}  // namespace

template <typename T>
cudaError_t potrf_lower(T* A, int64_t n, int64_t lda, T* dinv, int32_t* status_dev, cudaStream_t stream) {
  constexpr bool acc64 = sizeof(T) == 8;
  cudaError_t pe = prepare_diag_kernel<T>();
  if (pe != cudaSuccess) return pe;
  for (int64_t k0 = 0; k0 < n; k0 += NB) {
    const int nb = (int)((n - k0 < NB) ? (n - k0) : NB);
    T* Akk = A + k0 * lda + k0;
    T* dk = dinv + (k0 / NB) * NB * NB;
    count_launch();
    chol_diag_kernel<T><<<1, 256, diag_smem_bytes<T>(), stream>>>(Akk, lda, nb, dk, k0, status_dev);
    const int64_t rem = n - k0 - nb;
    if (rem <= 0) break;
    T* A21 = A + (k0 + nb) * lda + k0;
    T* A22 = A + (k0 + nb) * lda + (k0 + nb);
    // L21 = A21 inv(L11)^T.  In place: one thread block of the GEMM covers all nb (<= tile width) columns of its
    // rows and finishes reading them before it writes.
    cudaError_t e = gemm_simt(rem, nb, nb, 1.0, op<T>(A21, lda, 1), op<T>(dk, 1, NB), 0.0, op<T>(A21, lda, 1),
                              out<T>(A21, lda), false, acc64, stream);
    if (e != cudaSuccess) return e;
    // A22 -= L21 L21^T on the lower triangle
    e = gemm_simt(rem, rem, nb, -1.0, op<T>(A21, lda, 1), op<T>(A21, 1, lda), 1.0, op<T>(A22, lda, 1),
                  out<T>(A22, lda), true, acc64, stream);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

template <typename T>
cudaError_t potrs_right(T* X, int64_t m, int64_t n, int64_t ldx, const T* L, int64_t ldl, const T* dinv,
                        cudaStream_t stream) {
  constexpr bool acc64 = sizeof(T) == 8;
  cudaError_t e;
  // Y L^T = X, block columns left to right
  for (int64_t j0 = 0; j0 < n; j0 += NB) {
    const int nb = (int)((n - j0 < NB) ? (n - j0) : NB);
    const T* dj = dinv + (j0 / NB) * NB * NB;
    T* Xj = X + j0;
    // Y_j = X_j inv(L_jj)^T : B(k, c) = dinv[c, k]
    e = gemm_simt(m, nb, nb, 1.0, op<T>(Xj, ldx, 1), op<T>(dj, 1, NB), 0.0, op<T>(Xj, ldx, 1), out<T>(Xj, ldx),
                  false, acc64, stream);
    if (e != cudaSuccess) return e;
    const int64_t rem = n - j0 - nb;
    if (rem > 0) {
      // X[:, j1:] -= Y_j L[j1:, j0:j0+nb]^T : B(k, c) = L[j1 + c, j0 + k]
      const T* Lb = L + (j0 + nb) * ldl + j0;
      T* Xr = X + j0 + nb;
      e = gemm_simt(m, rem, nb, -1.0, op<T>(Xj, ldx, 1), op<T>(Lb, 1, ldl), 1.0, op<T>(Xr, ldx, 1),
                    out<T>(Xr, ldx), false, acc64, stream);
      if (e != cudaSuccess) return e;
    }
  }
  // W L = Y, block columns right to left
  const int64_t nblk = ceil_div(n, NB);
  for (int64_t jb = nblk - 1; jb >= 0; --jb) {
    const int64_t j0 = jb * NB;
    const int nb = (int)((n - j0 < NB) ? (n - j0) : NB);
    const T* dj = dinv + jb * NB * NB;
    T* Xj = X + j0;
    // W_j = Y_j inv(L_jj) : B(k, c) = dinv[k, c]
    e = gemm_simt(m, nb, nb, 1.0, op<T>(Xj, ldx, 1), op<T>(dj, NB, 1), 0.0, op<T>(Xj, ldx, 1), out<T>(Xj, ldx),
                  false, acc64, stream);
    if (e != cudaSuccess) return e;
    if (j0 > 0) {
      // Y[:, :j0] -= W_j L[j0:j0+nb, :j0] : B(k, c) = L[j0 + k, c]
      const T* Lb = L + j0 * ldl;
      e = gemm_simt(m, j0, nb, -1.0, op<T>(Xj, ldx, 1), op<T>(Lb, ldl, 1), 1.0, op<T>(X, ldx, 1), out<T>(X, ldx),
                    false, acc64, stream);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaGetLastError();
}

template cudaError_t potrf_lower<float>(float*, int64_t, int64_t, float*, int32_t*, cudaStream_t);
template cudaError_t potrf_lower<double>(double*, int64_t, int64_t, double*, int32_t*, cudaStream_t);
template cudaError_t potrs_right<float>(float*, int64_t, int64_t, int64_t, const float*, int64_t, const float*,
                                        cudaStream_t);
template cudaError_t potrs_right<double>(double*, int64_t, int64_t, int64_t, const double*, int64_t, const double*,
                                         cudaStream_t);

}  // namespace sp
