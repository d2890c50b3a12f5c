// Strided CUDA-core GEMM: the fp32-mode contraction kernel (fp32 storage, fp64 accumulation) and the workhorse of
// the blocked Cholesky / triangular solves.  Operand element types are chosen at run time; the accumulator type and
// the tile shape are compile-time.
#include "sp_common.cuh"

namespace sp {
namespace {

template <typename Acc>
__device__ __forceinline__ Acc load_elem(const void* p, int32_t dt, int64_t idx) {
  switch (dt) {
    case SP_BF16: return (Acc)__bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
    case SP_F64: return (Acc) reinterpret_cast<const double*>(p)[idx];
    default: return (Acc) reinterpret_cast<const float*>(p)[idx];
  }
}

template <typename Acc>
__device__ __forceinline__ void store_elem(void* p, int32_t dt, int64_t idx, Acc v) {
  switch (dt) {
    case SP_BF16: reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn((float)v); break;
    case SP_F64: reinterpret_cast<double*>(p)[idx] = (double)v; break;
    default: reinterpret_cast<float*>(p)[idx] = (float)v; break;
  }
}

constexpr int BK = 16;

template <typename Acc, int BM, int BN, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
gemm_simt_kernel(int64_t M, int64_t N, int64_t K, Acc alpha, Operand A, Operand B, Acc beta, Operand Cin,
                 OutOperand C, int lower_only) {
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int EA = BM * BK / NT;
  constexpr int EB = BN * BK / NT;
  static_assert(BM * BK % NT == 0 && BN * BK % NT == 0, "tile / thread mismatch");

  const int64_t row0 = (int64_t)blockIdx.y * BM;
  const int64_t col0 = (int64_t)blockIdx.x * BN;
  if (lower_only && row0 + BM - 1 < col0) return;

  __shared__ Acc As[BK][BM + 4];
  __shared__ Acc Bs[BK][BN + 4];

  const int t = threadIdx.x;
  const int tx = t % (BN / TN);
  const int ty = t / (BN / TN);
  const bool a_kfast = (A.s1 == 1);
  const bool b_nfast = (B.s1 == 1);

  Acc acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = (Acc)0;

  Acc ra[EA], rb[EB];

  auto fetch = [&](int64_t k0) {
#pragma unroll
    for (int r = 0; r < EA; ++r) {
      const int e = t + r * NT;
      const int i = a_kfast ? e / BK : e % BM;
      const int k = a_kfast ? e % BK : e / BM;
      const int64_t gi = row0 + i, gk = k0 + k;
      ra[r] = (gi < M && gk < K) ? load_elem<Acc>(A.ptr, A.dtype, gi * A.s0 + gk * A.s1) : (Acc)0;
    }
#pragma unroll
    for (int r = 0; r < EB; ++r) {
      const int e = t + r * NT;
      const int j = b_nfast ? e % BN : e / BK;
      const int k = b_nfast ? e / BN : e % BK;
      const int64_t gj = col0 + j, gk = k0 + k;
      rb[r] = (gj < N && gk < K) ? load_elem<Acc>(B.ptr, B.dtype, gk * B.s0 + gj * B.s1) : (Acc)0;
    }
  };

  fetch(0);
  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    __syncthreads();
#pragma unroll
    for (int r = 0; r < EA; ++r) {
      const int e = t + r * NT;
      const int i = a_kfast ? e / BK : e % BM;
      const int k = a_kfast ? e % BK : e / BM;
      As[k][i] = ra[r];
    }
#pragma unroll
    for (int r = 0; r < EB; ++r) {
      const int e = t + r * NT;
      const int j = b_nfast ? e % BN : e / BK;
      const int k = b_nfast ? e / BN : e % BK;
      Bs[k][j] = rb[r];
    }
    __syncthreads();
    if (k0 + BK < K) fetch(k0 + BK);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      Acc av[TM], bv[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) av[i] = As[k][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) bv[j] = Bs[k][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] += av[i] * bv[j];
    }
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t gi = row0 + ty * TM + i;
    if (gi >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int64_t gj = col0 + tx * TN + j;
      if (gj >= N) continue;
      Acc v = alpha * acc[i][j];
      if (beta != (Acc)0) v += beta * load_elem<Acc>(Cin.ptr, Cin.dtype, gi * Cin.s0 + gj * Cin.s1);
      store_elem<Acc>(C.ptr, C.dtype, gi * C.ld + gj, v);
    }
  }
}

}  // namespace

cudaError_t gemm_simt(int64_t M, int64_t N, int64_t K, double alpha, Operand A, Operand B, double beta, Operand Cin,
                      OutOperand C, bool lower_only, bool acc64, cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  count_launch();
  ProfScope prof(PK_GEMM_SIMT, (lower_only ? 1.0 : 2.0) * (double)M * (double)N * (double)K, 0.0, stream);
  if (acc64) {
    constexpr int BM = 64, BN = 64;
    dim3 grid((unsigned)ceil_div(N, BN), (unsigned)ceil_div(M, BM));
    gemm_simt_kernel<double, BM, BN, 4, 4><<<grid, 256, 0, stream>>>(M, N, K, alpha, A, B, beta, Cin, C,
                                                                      lower_only ? 1 : 0);
  } else {
    constexpr int BM = 128, BN = 128;
    dim3 grid((unsigned)ceil_div(N, BN), (unsigned)ceil_div(M, BM));
    gemm_simt_kernel<float, BM, BN, 8, 8><<<grid, 256, 0, stream>>>(M, N, K, (float)alpha, A, B, (float)beta, Cin, C,
                                                                     lower_only ? 1 : 0);
  }
  return cudaGetLastError();
}

}  // namespace sp
