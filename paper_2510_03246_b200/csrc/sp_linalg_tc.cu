// fp32 Cholesky factorisation and triangular solves whose O(n^3) / O(m n^2) work runs on the tensor cores.
//
// The regularised weight recovery W = R (G + rho I)^-1 needs fp32-level accuracy (G is a Gram matrix of ReLU
// activations with a condition number of the order of its size), which a plain bf16 product cannot give.  Every fp32
// value is therefore held as an exact sum of three bf16 parts (hi + mid + lo, 3 x 8 mantissa bits), and a product
// of two such operands is taken as the six part products of weight >= 2^-16 (hi.hi, hi.mid, mid.hi, hi.lo, lo.hi,
// mid.mid), each a K segment of one tcgen05 GEMM with fp32 accumulation.  The dropped terms are below 2^-23.
//
// Blocked right-looking algorithm with 128-wide panels:
//   diagonal block : one CTA factorises it in registers (4 x 4 elements per thread, four columns per step) and forms
//                    inv(L11) in the same sweep (the row operations of the elimination applied to an identity block);
//   panel          : L21 = A21 inv(L11)^T on the CUDA cores (K = 128), written as fp32 and as the three bf16 parts;
//   trailing update: A22 -= L21 L21^T (lower triangle) as one six-segment tensor-core GEMM.
// The triangular solves X L^T = R, W L = X use the same two kernels block column by block column.
#include "sp_common.cuh"

namespace sp {
namespace {

constexpr int TB = kCholTcNB;          // 128
constexpr int DIAG_BLOCKS = (TB / 4) * (TB / 4 + 1) / 2;   // 528 lower-triangular 4 x 4 blocks
constexpr int DIAG_THREADS = 544;      // 17 warps

// 1 / sqrt(x) to about 1 ulp: hardware approximation plus one Newton step.
__device__ __forceinline__ float rsqrt_refined(float x) {
  float r;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r * fmaf(-0.5f * x, r * r, 1.5f);
}

constexpr int DIAG_TPAD = TB + 1;
constexpr size_t DIAG_SMEM = (size_t)TB * DIAG_TPAD * sizeof(float);

// Factorise the nb x nb diagonal block at A (lower triangle, left as it is) and write inv(L) and its transpose to
// dinv[0 : TB*TB] and dinv[TB*TB : 2*TB*TB] (row-major TB x TB, zero above / below the diagonal respectively,
// identity on the padding rows nb..TB-1).  A non-positive pivot is reported once through `status` and replaced by 1.
//
// One thread owns one 4 x 4 block (bi, bj), bj <= bi, of the lower triangle in registers.  Blocked right-looking
// elimination, four columns per step jb, that carries inv(L) along (the row operations of the elimination applied to
// an identity block B).  Register block m holds the trailing matrix on block columns > jb and B on block columns
// <= jb; a block column of the trailing matrix is final when its step comes and moves to lcol.  Per step:
//   1. the owner of the diagonal block factorises it, D = C C^T, and inverts C (sequential, one thread; it runs while
//      the other threads still finish step jb - 1);
//   2. owners of block column jb:  L_i = A_i C^-T (final);  owners of block row jb:  B_jb <- C^-1 B_jb (final rows of
//      inv(L)).  Both go to the shared array W (4 values per index): W[:, i] = L[i, j0:j0+4] for rows below the
//      block, W[:, c] = inv(L)[j0:j0+4, c] for columns up to the block;
//   3. every block below block row jb:  m -= W[:, rows]^T W[:, cols]  — the trailing update where the block still
//      holds the matrix, the update of B where it holds B (a block of block column jb starts its life as B from 0).
// Global input and output go through a padded shared tile so that every global access is a full coalesced row.
__global__ void __launch_bounds__(DIAG_THREADS) chol_diag128_kernel(float* A, int64_t lda, int nb, float* dinv,
                                                                    int64_t row0, int32_t* status,
                                                                    const int32_t* skip, int64_t a_bs, int64_t d_bs) {
  if (skip != nullptr && *skip != 0) return;                  // conditional launch (see SkipScope)
  A += (int64_t)blockIdx.x * a_bs;                            // batched launch: one CTA per system
  dinv += (int64_t)blockIdx.x * d_bs;
  extern __shared__ __align__(16) float diag_tile[];          // T[TB][TB + 1]
  float (*T)[DIAG_TPAD] = reinterpret_cast<float (*)[DIAG_TPAD]>(diag_tile);
  __shared__ __align__(16) float W[2][4][TB];   // W[k][index]: conflict-free 16-byte accesses along the index
  __shared__ __align__(16) float Ci_s[2][16];   // inverse of the diagonal factor, row-major 4 x 4 (lower)
  const int t = threadIdx.x;
  const int lane = t & 31, warp = t >> 5;
  constexpr int NWARP = DIAG_THREADS / 32;
  const bool active = t < DIAG_BLOCKS;
  // t = bi (bi + 1) / 2 + bj with bj <= bi
  int bi = (int)((sqrtf(8.f * (float)t + 1.f) - 1.f) * 0.5f);
  while ((bi + 1) * (bi + 2) / 2 <= t) ++bi;
  while (bi * (bi + 1) / 2 > t) --bi;
  const int bj = t - bi * (bi + 1) / 2;

  // ---- load: one warp per row, lanes along the columns; identity on the padding
  for (int i = warp; i < TB; i += NWARP)
    for (int c = lane; c < TB; c += 32) {
      float v = 0.f;
      if (i < nb && c <= i) v = A[(int64_t)i * lda + c];
      if (i >= nb && i == c) v = 1.f;
      T[i][c] = v;
    }
  __syncthreads();
  float m[4][4], lcol[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      m[r][s] = active ? T[4 * bi + r][4 * bj + s] : 0.f;
      lcol[r][s] = 0.f;
    }

  // step 1 for block jb by its diagonal owner: C -> lcol, C^-1 -> m, shared copies of C^-1
  auto factor_diag = [&](int jb) {
    float c[4][4], ci[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int s = 0; s < 4; ++s) { c[r][s] = 0.f; ci[r][s] = 0.f; }
    float rd[4];   // reciprocals of the diagonal of C
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float p = m[k][k];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (q < k) p = fmaf(-c[k][q], c[k][q], p);
      if (!(p > 0.f)) {
        report_status(status, SP_ERR_NOT_SPD, (int32_t)(row0 + 4 * jb + k), 0);
        p = 1.f;
      }
      rd[k] = rsqrt_refined(p);
      c[k][k] = p * rd[k];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        if (r > k) {
          float v = m[r][k];
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (q < k) v = fmaf(-c[r][q], c[k][q], v);
          c[r][k] = v * rd[k];
        }
      }
    }
    // inverse of the lower-triangular C by forward substitution, column by column
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      ci[s][s] = rd[s];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        if (r > s) {
          float v = 0.f;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (q >= s && q < r) v = fmaf(c[r][q], ci[q][s], v);
          ci[r][s] = -v * rd[r];
        }
      }
    }
    float* cs = Ci_s[jb & 1];
    float (*w)[TB] = W[jb & 1];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        lcol[r][s] = c[r][s];
        m[r][s] = ci[r][s];
        cs[r * 4 + s] = ci[r][s];
        w[r][4 * jb + s] = ci[r][s];          // W[k][c] = inv(L)[j0 + k][c]
      }
  };

  if (active && bi == 0) factor_diag(0);
  const int nsteps = (nb + 3) / 4;
  for (int jb = 0; jb < nsteps; ++jb) {
    float (*w)[TB] = W[jb & 1];
    __syncthreads();
    if (active && bj == jb && bi > jb) {
      // L_i = A_i C^-T : L_i[r][k] = sum_{s <= k} A_i[r][s] Ci[k][s]
      const float* cs = Ci_s[jb & 1];
      float l[4][4];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float v = 0.f;
#pragma unroll
          for (int s2 = 0; s2 < 4; ++s2)
            if (s2 <= k) v = fmaf(m[r][s2], cs[k * 4 + s2], v);
          l[r][k] = v;
        }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        *reinterpret_cast<float4*>(&w[k][4 * bi]) = make_float4(l[0][k], l[1][k], l[2][k], l[3][k]);
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int k = 0; k < 4; ++k) { lcol[r][k] = l[r][k]; m[r][k] = 0.f; }
    }
    if (active && bi == jb && bj < jb) {
      // B_jb <- C^-1 B_jb : Bn[k][s] = sum_{r <= k} Ci[k][r] B[r][s]
      const float* cs = Ci_s[jb & 1];
      float bn[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) {
          float v = 0.f;
#pragma unroll
          for (int r = 0; r < 4; ++r)
            if (r <= k) v = fmaf(cs[k * 4 + r], m[r][s2], v);
          bn[k][s2] = v;
        }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        *reinterpret_cast<float4*>(&w[k][4 * bj]) = make_float4(bn[k][0], bn[k][1], bn[k][2], bn[k][3]);
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) m[k][s2] = bn[k][s2];
      }
    }
    __syncthreads();
    if (active && bi > jb) {
      float wr[4][4], wc[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 v = *reinterpret_cast<const float4*>(&w[k][4 * bi]);
        wr[0][k] = v.x; wr[1][k] = v.y; wr[2][k] = v.z; wr[3][k] = v.w;
        const float4 u = *reinterpret_cast<const float4*>(&w[k][4 * bj]);
        wc[0][k] = u.x; wc[1][k] = u.y; wc[2][k] = u.z; wc[3][k] = u.w;
      }
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) {
          float v = m[r][s2];
#pragma unroll
          for (int k = 0; k < 4; ++k) v = fmaf(-wr[r][k], wc[s2][k], v);
          m[r][s2] = v;
        }
      // the owner of the next diagonal block goes straight on to factorise it
      if (bi == jb + 1 && bj == jb + 1 && jb + 1 < nsteps) factor_diag(jb + 1);
    }
  }

  // ---- store inv(L) and its transpose through the tile
  __syncthreads();
  for (int e = t; e < TB * TB; e += DIAG_THREADS) T[e / TB][e % TB] = 0.f;
  __syncthreads();
  if (active) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int s = 0; s < 4; ++s)
        if (4 * bj + s <= 4 * bi + r) T[4 * bi + r][4 * bj + s] = m[r][s];
  }
  __syncthreads();
  for (int i = warp; i < TB; i += NWARP)
    for (int c = lane; c < TB; c += 32) {
      dinv[i * TB + c] = T[i][c];
      dinv[TB * TB + i * TB + c] = T[c][i];      // row i of the transpose = column i of inv(L)
    }
  // L itself is not written back: the solves use inv(L) of the diagonal blocks and the blocks of L below them only.
  (void)lcol;
}

__device__ __forceinline__ void split3(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(hi);
  mid = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(mid);
  lo = __float2bfloat16_rn(r2);
}

// ---- staging of one 128 x 128 fp32 block (64 KiB) into shared memory by bulk asynchronous copies
__device__ __forceinline__ uint32_t lin_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// One thread: arm the barrier with the byte count and issue the copies (four of 16 KiB).
__device__ __forceinline__ void stage_block_issue(float* dst_smem, const float* src, uint64_t* bar) {
  const uint32_t b = lin_smem_u32(bar);
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)(TB * TB * 4))
               : "memory");
#pragma unroll
  for (int q = 0; q < 4; ++q)
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(lin_smem_u32(dst_smem + q * (TB * TB / 4))), "l"(src + q * (TB * TB / 4)),
                   "r"((uint32_t)(TB * TB)), "r"(b)
                 : "memory");
}
__device__ __forceinline__ void stage_bar_init(uint64_t* bar) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(lin_smem_u32(bar)) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Every thread: wait for the block (phase `parity`), at most about a second.  Returns false when the wait ran out.
__device__ __forceinline__ bool stage_block_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t b = lin_smem_u32(bar);
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(b), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((it & 0xffu) == 0xffu && clock64() - t0 > 2000000000ll) return false;
  }
}

constexpr int PA_ROWS = 32;
constexpr int PA_THREADS = 256;
constexpr int PA_APAD = PA_ROWS + 4;
constexpr size_t PA_SMEM = ((size_t)TB * TB + (size_t)TB * PA_APAD) * sizeof(float) + 128;
constexpr size_t PA_SMEM_NEAR = PA_SMEM + (size_t)TB * TB * sizeof(float);   // + the block of L of the second product

// Optional second product of the same launch (backward triangular solve, TRANS form only): with W_j the block column
// just computed, X[:, near columns] -= W_j L[j rows, near columns], the update of the block column the NEXT step
// needs, so that the chain of a solve is one kernel per block column.  L: fp32 factor, pointer to its element
// (first row of block j, first near column), leading dimension ldl (a multiple of 4, 16-byte aligned rows); Xn: first
// near column of X.  The far columns are updated by a tensor-core GEMM on another stream, which may still be adding
// into the near columns when this kernel runs: both add atomically.
struct PanelNear {
  const float* L;    // nullptr: no second product
  int64_t ldl;
  float* Xn;
};
// Batched launch of the panel kernel (grid.y = systems): element strides between the systems' arrays
struct PanelBatch {
  int64_t x = 0, dinv = 0, s = 0, near_l = 0;    // X (and the near columns), dinv, S, near.L
};

// X[i, 0:nb] <- X[i, 0:nb] inv(L)^T (TRANS == false) or X[i, 0:nb] inv(L) (TRANS == true), for `rows` rows.
// dinv is the pair of TB x TB blocks written by chol_diag128_kernel.  The result is written back in fp32 (write_f32)
// and as three bf16 parts to S[i * lds + part * s_seg + c] for all TB columns (zero beyond nb).
// One CTA takes 32 rows.  The 64 KiB block of inv(L) comes in by bulk copies while the threads fetch and transpose
// the rows of X; a thread then computes 4 rows x 4 columns (a warp: 4 rows x 128 columns).
template <bool TRANS>
__global__ void __launch_bounds__(PA_THREADS) panel_apply_kernel(float* X, int64_t ldx, int64_t rows, int nb,
                                                                 const float* __restrict__ dinv, __nv_bfloat16* S,
                                                                 int64_t lds, int64_t s_seg, int write_f32,
                                                                 int32_t* status, PanelNear near,
                                                                 const int32_t* skip, PanelBatch pb) {
  if (skip != nullptr && *skip != 0) return;
  X += (int64_t)blockIdx.y * pb.x;
  dinv += (int64_t)blockIdx.y * pb.dinv;
  if (S) S += (int64_t)blockIdx.y * pb.s;
  if (near.L) { near.L += (int64_t)blockIdx.y * pb.near_l; near.Xn += (int64_t)blockIdx.y * pb.x; }
  extern __shared__ __align__(128) float pa_smem[];
  float (*Lt)[TB] = reinterpret_cast<float (*)[TB]>(pa_smem);                       // Lt[k][c]
  float (*At)[PA_APAD] = reinterpret_cast<float (*)[PA_APAD]>(pa_smem + TB * TB);   // At[k][row]
  uint64_t* bar = reinterpret_cast<uint64_t*>(pa_smem + TB * TB + TB * PA_APAD);    // [0]: Lt landed, [1]: Bn landed
  float (*Bn)[TB] = reinterpret_cast<float (*)[TB]>(pa_smem + TB * TB + TB * PA_APAD + 32);   // Bn[k][c] (near only)
  const int t = threadIdx.x;
  const int64_t r0 = (int64_t)blockIdx.x * PA_ROWS;
  const bool x_al = (ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0);
  const bool do_near = TRANS && near.L != nullptr;
  if (t == 0) {
    stage_bar_init(bar);
    if (do_near) stage_bar_init(bar + 1);
  }
  __syncthreads();
  // Lt[k][c] = inv(L)[c][k] (the transposed copy) or inv(L)[k][c]: a straight copy either way
  if (t == 0) stage_block_issue(pa_smem, dinv + (TRANS ? 0 : TB * TB), bar);
  if (do_near && t < 32) {
    // rows j0 .. j0 + nb - 1 of L, TB columns each (512 bytes per row), one bulk copy per row, four per lane
    const uint32_t b1 = lin_smem_u32(bar + 1);
    if (t == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b1), "r"((uint32_t)(nb * TB * 4))
                   : "memory");
    __syncwarp();
    for (int k = t; k < nb; k += 32)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(lin_smem_u32(&Bn[k][0])), "l"(near.L + (int64_t)k * near.ldl), "r"((uint32_t)(TB * 4)),
                     "r"(b1)
                   : "memory");
  }
  {
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
#pragma unroll
    for (int q = 0; q < PA_ROWS * TB / 4 / PA_THREADS; ++q) {
      const int e = t + q * PA_THREADS;
      const int i = e / (TB / 4), k = (e % (TB / 4)) * 4;
      At[k][i] = xv[q].x; At[k + 1][i] = xv[q].y; At[k + 2][i] = xv[q].z; At[k + 3][i] = xv[q].w;
    }
  }
  // (the outcome is made uniform over the block: a thread whose wait ran out must not leave while others go on)
  const bool staged = __syncthreads_and(stage_block_wait(bar, 0) ? 1 : 0) != 0;
  if (!staged) {   // the copies did not land in time: report and leave X untouched
    if (t == 0) report_status(status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 10);
    return;
  }
  const int tx = t & 31, ty = t >> 5;   // columns 4 tx .. 4 tx + 3, rows 4 ty .. 4 ty + 3
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[r][j] = 0.f;
#pragma unroll 8
  for (int k = 0; k < TB; ++k) {
    const float4 a0 = *reinterpret_cast<const float4*>(&At[k][4 * ty]);
    const float4 l0 = *reinterpret_cast<const float4*>(&Lt[k][4 * tx]);
    const float av[4] = {a0.x, a0.y, a0.z, a0.w};
    const float lv[4] = {l0.x, l0.y, l0.z, l0.w};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
  }
  const bool x_vec = write_f32 && x_al;
  const int c0 = 4 * tx;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int64_t gi = r0 + 4 * ty + r;
    if (gi >= rows) continue;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = (c0 + j < nb) ? acc[r][j] : 0.f;
    if (write_f32) {
      float* dst = X + gi * ldx + c0;
      if (x_vec && c0 + 4 <= nb) {
        *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (c0 + j < nb) dst[j] = v[j];
      }
    }
    if (S) {   // S + gi * lds + part * s_seg + c0 is 8-byte aligned by construction (lds, s_seg multiples of 8)
      __align__(8) __nv_bfloat16 part[3][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) split3(v[j], part[0][j], part[1][j], part[2][j]);
#pragma unroll
      for (int q = 0; q < 3; ++q)
        *reinterpret_cast<uint2*>(S + gi * lds + q * s_seg + c0) = *reinterpret_cast<const uint2*>(part[q]);
    }
  }

  if (do_near) {
    // ---- second product: X[rows, near columns] -= W_j Bn.  W_j goes back to shared memory as the left operand
    // (At[k][row], k = column of W_j); rows of Bn beyond nb are cleared by hand (no copy wrote them).
    __syncthreads();     // everyone is done reading At
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int j = 0; j < 4; ++j) At[c0 + j][4 * ty + r] = (c0 + j < nb) ? acc[r][j] : 0.f;
    for (int e = t; e < (TB - nb) * TB; e += PA_THREADS) Bn[nb + e / TB][e % TB] = 0.f;
    const bool staged2 = __syncthreads_and(stage_block_wait(bar + 1, 0) ? 1 : 0) != 0;
    if (!staged2) {
      if (t == 0) report_status(status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 12);
      return;
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[r][j] = 0.f;
#pragma unroll 8
    for (int k = 0; k < TB; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&At[k][4 * ty]);
      const float4 l0 = *reinterpret_cast<const float4*>(&Bn[k][4 * tx]);
      const float av[4] = {a0.x, a0.y, a0.z, a0.w};
      const float lv[4] = {l0.x, l0.y, l0.z, l0.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int64_t gi = r0 + 4 * ty + r;
      if (gi >= rows) continue;
      float* dst = near.Xn + gi * ldx + c0;      // 16-byte aligned: the launcher checks ldx and the base
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(-acc[r][0]), "f"(-acc[r][1]),
                   "f"(-acc[r][2]), "f"(-acc[r][3])
                   : "memory");
    }
  }
}

template <bool TRANS>
cudaError_t launch_panel_apply(float* X, int64_t ldx, int64_t rows, int nb, const float* dinv, __nv_bfloat16* S,
                               int64_t lds, int64_t s_seg, bool write_f32, int32_t* status, cudaStream_t stream,
                               PanelNear near = PanelNear{nullptr, 0, nullptr}, int batch = 1,
                               PanelBatch pb = PanelBatch{}) {
  static PerDeviceOnce attr_once;      // one per instantiation; the attribute belongs to the device's context
  {
    cudaError_t e = attr_once.run([] {
      return cudaFuncSetAttribute(panel_apply_kernel<TRANS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)PA_SMEM_NEAR);
    });
    if (e != cudaSuccess) return e;
  }
  if (rows <= 0) return cudaSuccess;
  count_launch();
  const bool with_near = TRANS && near.L != nullptr;
  ProfScope prof(PK_PANEL_APPLY, (with_near ? 4.0 : 2.0) * (double)rows * TB * TB, 0.0, stream);
  panel_apply_kernel<TRANS><<<dim3((unsigned)ceil_div(rows, PA_ROWS), (unsigned)batch), PA_THREADS,
                              with_near ? PA_SMEM_NEAR : PA_SMEM, stream>>>(
      X, ldx, rows, nb, dinv, S, lds, s_seg, write_f32 ? 1 : 0, status, near, skip_flag(), pb);
  return cudaGetLastError();
}

// The six kept part products of two three-part operands: A parts (hi, hi, mid, hi, lo, mid) against B parts
// (hi, mid, hi, lo, hi, mid).
// ---------------------------------------------------------------------------------------------------------------
// Lookahead of the factorisation: the NEXT diagonal block, updated with the block column just factored, in one small
// launch, so that its factorisation does not wait for the full panel and the trailing update:
//   Lm = A21 inv(L_kk)^T  (nb2 x 128),   S = A22 - Lm Lm^T  (nb2 x nb2, fp32, into a scratch block with ld 128)
// with A21 = A[next block rows, block k columns] and A22 = A[next block, next block] as the trailing updates up to
// step k - 1 left them.  One cluster of 8 CTAs, 16 rows each: every CTA forms its rows of Lm, publishes them
// (transposed, in global scratch LmT[c][row]), the cluster meets, and every CTA forms its rows of S from all of Lm.
constexpr int NM_ROWS = 16, NM_THREADS = 256, NM_APAD = NM_ROWS + 4, NM_CTAS = TB / NM_ROWS;
constexpr size_t NM_SMEM = ((size_t)TB * TB + (size_t)TB * NM_APAD) * sizeof(float) + 16;
static_assert(NM_CTAS == 8, "one portable cluster covers the block");

__device__ __forceinline__ void cluster_meet() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// MODE 0: both stages in one launch, the CTAs being one cluster (they meet between the stages);
// MODE 1 / MODE 2: the stages as two launches of 8 independent CTAs (for use beside persistent GEMM CTAs that hold
// most SMs, where a cluster of 8 waits for a free group of SMs).
template <int MODE>
__device__ __forceinline__ void next_diag_body(const float* __restrict__ A21, const float* __restrict__ A22,
                                               int64_t lda, int nb2, const float* __restrict__ dinv, float* LmT,
                                               float* S, int32_t* status) {
  extern __shared__ __align__(128) float nm_smem[];
  float (*Lt)[TB] = reinterpret_cast<float (*)[TB]>(nm_smem);                       // Lt[k][c]
  float (*At)[NM_APAD] = reinterpret_cast<float (*)[NM_APAD]>(nm_smem + TB * TB);   // At[k][row]
  uint64_t* bar = reinterpret_cast<uint64_t*>(nm_smem + TB * TB + TB * NM_APAD);
  const int t = threadIdx.x;
  const int i0 = (int)blockIdx.x * NM_ROWS;
  const int tx = t & 31, ty = t >> 5;   // columns 4 tx .. 4 tx + 3; rows 2 ty, 2 ty + 1
  float acc[2][4];
  if (MODE != 2) {
    // ---- stage 1: rows i0 .. i0 + 15 of Lm; Lt[k][c] = inv(L)[c][k] comes in by bulk copies
    if (t == 0) stage_bar_init(bar);
    __syncthreads();
    if (t == 0) stage_block_issue(nm_smem, dinv + TB * TB, bar);
    for (int e = t; e < NM_ROWS * TB; e += NM_THREADS) {
      const int i = e / TB, k = e % TB;
      At[k][i] = (i0 + i < nb2) ? A21[(int64_t)(i0 + i) * lda + k] : 0.f;
    }
    const bool staged = __syncthreads_and(stage_block_wait(bar, 0) ? 1 : 0) != 0;
    if (!staged && t == 0) report_status(status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 11);
    // (a CTA whose copies did not land still goes on to the barrier below; its rows are then wrong and the status
    //  says so)
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[r][j] = 0.f;
#pragma unroll 8
    for (int k = 0; k < TB; ++k) {
      const float2 a = *reinterpret_cast<const float2*>(&At[k][2 * ty]);
      const float4 l0 = *reinterpret_cast<const float4*>(&Lt[k][4 * tx]);
      const float av[2] = {a.x, a.y};
      const float lv[4] = {l0.x, l0.y, l0.z, l0.w};
#pragma unroll
      for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
    }
    __syncthreads();   // everyone is done with At and Lt
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = 4 * tx + j;
      const float2 v = make_float2(acc[0][j], acc[1][j]);
      *reinterpret_cast<float2*>(&At[c][2 * ty]) = v;                              // own rows, left operand of stage 2
      *reinterpret_cast<float2*>(&LmT[(int64_t)c * TB + i0 + 2 * ty]) = v;         // for the other CTAs
    }
    if (MODE == 1) return;
    cluster_meet();
  }
  // ---- stage 2: rows i0 .. i0 + 15 of S; Lt[c][j] = Lm[j][c]
  {
    const float4* src = reinterpret_cast<const float4*>(LmT);
    float4* dst = reinterpret_cast<float4*>(nm_smem);
#pragma unroll
    for (int q = 0; q < TB * TB / 4 / NM_THREADS; ++q) dst[t + q * NM_THREADS] = __ldcg(src + t + q * NM_THREADS);
    if (MODE == 2)     // own rows of Lm come from the first launch
      for (int e = t; e < NM_ROWS * TB; e += NM_THREADS) {
        const int c = e / NM_ROWS, i = e % NM_ROWS;
        At[c][i] = __ldcg(&LmT[(int64_t)c * TB + i0 + i]);
      }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[r][j] = 0.f;
#pragma unroll 8
  for (int k = 0; k < TB; ++k) {
    const float2 a = *reinterpret_cast<const float2*>(&At[k][2 * ty]);
    const float4 l0 = *reinterpret_cast<const float4*>(&Lt[k][4 * tx]);
    const float av[2] = {a.x, a.y};
    const float lv[4] = {l0.x, l0.y, l0.z, l0.w};
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[r][j] = fmaf(av[r], lv[j], acc[r][j]);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int i = i0 + 2 * ty + r;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = 4 * tx + j;
      v[j] = (i < nb2 && c <= i) ? A22[(int64_t)i * lda + c] - acc[r][j] : 0.f;
    }
    *reinterpret_cast<float4*>(&S[i * TB + 4 * tx]) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

__global__ void __cluster_dims__(NM_CTAS, 1, 1) __launch_bounds__(NM_THREADS)
    chol_next_diag_kernel(const float* __restrict__ A21, const float* __restrict__ A22, int64_t lda, int nb2,
                          const float* __restrict__ dinv, float* LmT, float* S, int32_t* status,
                          const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  next_diag_body<0>(A21, A22, lda, nb2, dinv, LmT, S, status);
}
__global__ void __launch_bounds__(NM_THREADS)
    chol_next_diag_stage1_kernel(const float* __restrict__ A21, int64_t lda, int nb2, const float* __restrict__ dinv,
                                 float* LmT, int32_t* status, const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  next_diag_body<1>(A21, nullptr, lda, nb2, dinv, LmT, nullptr, status);
}
__global__ void __launch_bounds__(NM_THREADS)
    chol_next_diag_stage2_kernel(const float* __restrict__ A22, int64_t lda, int nb2, float* LmT, float* S,
                                 const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  next_diag_body<2>(nullptr, A22, lda, nb2, nullptr, LmT, S, nullptr);
}

// two-level blocking of the factorisation (see potrf_lower_tc): systems of at least kOuterMinN rows, outer blocks of
// kOuterBlocks diagonal blocks
constexpr int64_t kOuterMinN = 12288;
constexpr int64_t kOuterBlocks = 4;

constexpr int kPartA[6] = {0, 0, 1, 0, 2, 1};
constexpr int kPartB[6] = {0, 1, 0, 2, 0, 1};

}  // namespace

int64_t chol_tc_pad(int64_t n) { return (n + TB - 1) / TB * TB; }

sp_status potrf_lower_tc(float* A, int64_t n, int64_t lda, float* dinv, void* Pv, int32_t* status_dev,
                         cudaStream_t stream, const SolveAssist* assist, int64_t m_extra, bool split_lookahead) {
  __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(Pv);
  const int64_t np = chol_tc_pad(n), ldp = 3 * np;
  const int64_t nblk = ceil_div(n, (int64_t)TB);
  const int32_t* skip = skip_flag();
  static PerDeviceOnce attr_once;
  if (attr_once.run([] {
        cudaError_t e = cudaFuncSetAttribute(chol_diag128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)DIAG_SMEM);
        if (e == cudaSuccess)
          e = cudaFuncSetAttribute(chol_next_diag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)NM_SMEM);
        if (e == cudaSuccess)
          e = cudaFuncSetAttribute(chol_next_diag_stage1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)NM_SMEM);
        if (e == cudaSuccess)
          e = cudaFuncSetAttribute(chol_next_diag_stage2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)NM_SMEM);
        return e;
      }) != cudaSuccess)
    return SP_ERR_CUDA;
#define SP_CUDA_OK(x) do { if ((x) != cudaSuccess) return SP_ERR_CUDA; } while (0)
  // With an assisting stream the chain of diagonal blocks runs ahead: after block k is factored, a small kernel
  // forms the next diagonal block (into scratch behind the inverses), and the next factorisation starts from it while
  // the full panel and the trailing update of step k run on the assisting stream.
  float* S = dinv + nblk * 2 * TB * TB;      // [128, 128] next diagonal block
  float* LmT = S + TB * TB;                  // [128, 128] scratch of the lookahead kernel
  bool rec[2] = {false, false};
  // Far part of a step's trailing update on a stream of its own: it adds into the matrix through the GEMM's atomic TMA
  // reduction (which needs 16-byte aligned rows and a width that is a multiple of 4), so it commutes with the near
  // update of the next step, which touches one of its block columns.  What must see it complete waits for its event:
  // the lookahead kernel of step kb reads block (kb+1, kb+1), last touched by the far update of step kb - 2.
  // The far GEMM leaves a few SM pairs to the kernels of the chain, which would otherwise wait for its tiles to end.
  const bool far_apart = assist && assist->far_stream && n % 4 == 0 && lda % 4 == 0 &&
                         (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && !reproducible_mode();
  bool far_rec[2] = {false, false};
  constexpr int kFarPairs = 64;
  // Two-level blocking for large systems: the trailing update of a step is bound by the read-modify-write of the fp32
  // matrix when K is only 128 (n = 28672: 430 GB per factorisation).  With OB > 1 the steps of an outer block of OB
  // diagonal blocks update only the rest of that outer block's columns at once; everything to the right of it gets
  // ONE update per outer block with K = OB * 128, which divides that traffic by OB.
  const int64_t OB = (assist && n >= kOuterMinN) ? kOuterBlocks : 1;
  for (int64_t kb = 0; kb < nblk; ++kb) {
    const int64_t k0 = kb * TB;
    const int nb = (int)((n - k0 < TB) ? (n - k0) : TB);
    float* dk = dinv + kb * 2 * TB * TB;
    const int64_t ob_start = kb / OB * OB;
    const int64_t ob_end_blk = (ob_start + OB < nblk) ? ob_start + OB : nblk;
    const int64_t ob_end_col = (ob_end_blk * TB < n) ? ob_end_blk * TB : n;
    const bool outer = OB > 1;
    const bool inner_last = outer && kb == ob_end_blk - 1;
    const bool inner_first = outer && kb == ob_start;
    {
      // the first block of an outer block is read from the matrix itself, once the first columns of the previous
      // outer block's update have landed; every other block comes from the lookahead kernel's scratch
      const bool from_scratch = assist && kb > 0 && !inner_first;
      if (assist && inner_first && kb > 0) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->near_done, 0));
      count_launch();
      ProfScope prof(PK_CHOL_DIAG, (double)nb * nb * nb * (2.0 / 3.0), 0.0, stream);
      chol_diag128_kernel<<<1, DIAG_THREADS, DIAG_SMEM, stream>>>(from_scratch ? S : A + k0 * lda + k0,
                                                                  from_scratch ? (int64_t)TB : lda, nb, dk, k0,
                                                                  status_dev, skip, 0, 0);
      if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    }
    const int64_t rem = n - k0 - nb;
    // rows below the block that the panel covers: the rest of the matrix and the m_extra appended rows (right-hand
    // sides of a system X L^T = B stored below A: the panel and the trailing update are exactly their forward
    // substitution, so it costs no steps of its own)
    const int64_t prow = rem + m_extra;
    if (prow <= 0) break;
    cudaStream_t sb = stream;
    // last block with appended rows: their panel runs on `stream`, behind the assisting stream's last update
    if (assist && rem <= 0 && kb >= 1) {
      SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->rest_done[(kb - 1) & 1], 0));
      for (int q = 0; q < 2; ++q)
        if (far_rec[q]) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->far_done[q], 0));
    }
    if (assist && rem > 0) {
      if (!inner_last) {
        // next diagonal block: it reads blocks (kb+1, kb) and (kb+1, kb+1), i.e. the first two block columns of the
        // trailing update of step kb - 1, which that step issues first and signals on their own
        if (kb >= 1) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->near_done, 0));
        if (far_rec[kb & 1]) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->far_done[kb & 1], 0));   // far update of step kb - 2
        const int nb2 = (int)(rem < TB ? rem : TB);
        count_launch();
        ProfScope prof(PK_PANEL_APPLY, 4.0 * TB * TB * TB, 0.0, stream);
        if (!split_lookahead) {
          chol_next_diag_kernel<<<NM_CTAS, NM_THREADS, NM_SMEM, stream>>>(A + (k0 + nb) * lda + k0,
                                                                          A + (k0 + nb) * lda + (k0 + nb), lda, nb2,
                                                                          dk, LmT, S, status_dev, skip);
        } else {
          chol_next_diag_stage1_kernel<<<NM_CTAS, NM_THREADS, NM_SMEM, stream>>>(A + (k0 + nb) * lda + k0, lda, nb2, dk,
                                                                                 LmT, status_dev, skip);
          count_launch();
          chol_next_diag_stage2_kernel<<<NM_CTAS, NM_THREADS, NM_SMEM, stream>>>(A + (k0 + nb) * lda + (k0 + nb), lda,
                                                                                 nb2, LmT, S, skip);
        }
        if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
      }
      // the panel overwrites A21 in place: it starts behind the lookahead kernel
      SP_CUDA_OK(cudaEventRecord(assist->panel_done, stream));
      sb = assist->stream;
      SP_CUDA_OK(cudaStreamWaitEvent(sb, assist->panel_done, 0));
    }
    // L21 = A21 inv(L11)^T, fp32 in place and as bf16 parts in P[k0+nb.., part * np + k0 ..]
    if (launch_panel_apply<false>(A + (k0 + nb) * lda + k0, lda, prow, nb, dk, P + (k0 + nb) * ldp + k0, ldp, np, true,
                                  status_dev, sb) != cudaSuccess)
      return SP_ERR_CUDA;
    if (rem <= 0) break;     // last block: the appended rows are done, nothing is left to update
    if (far_apart && !outer && rem > 2 * TB) SP_CUDA_OK(cudaEventRecord(assist->far_go, sb));   // the panel's parts exist
    // A22 -= L21 L21^T on the lower triangle
    TcOperand ta{P + (k0 + nb) * ldp, ldp, true}, tb{P + (k0 + nb) * ldp, ldp, true};
    ta.kext = tb.kext = ldp;
    ta.mnext = prow;
    tb.mnext = rem;
    TcSegments sg;
    sg.nseg = 6;
    for (int q = 0; q < 6; ++q) {
      sg.a_k[q] = (int32_t)(kPartA[q] * np + k0);
      sg.b_k[q] = (int32_t)(kPartB[q] * np + k0);
    }
    float* A22 = A + (k0 + nb) * lda + (k0 + nb);
    constexpr int64_t kNear = 2 * TB;     // block columns of the update that the next step's chain kernels read
    if (outer) {
      // (a) the rest of this outer block's columns, all rows below: K = 128
      const int64_t cols_in = ob_end_col - (k0 + nb);
      if (cols_in > 0) {
        tb.mnext = cols_in;
        sp_status st = gemm_tc(prow, cols_in, TB, -1.f, ta, tb, 1.f, Operand{A22, SP_F32, lda, 1},
                               OutOperand{A22, SP_F32, lda}, true, status_dev, sb, &sg,
                               (2.0 * (double)prow * (double)cols_in - (double)cols_in * (double)cols_in) * (double)nb);
        if (st != SP_OK) return st;
        SP_CUDA_OK(cudaEventRecord(assist->near_done, sb));
      }
      // (b) after the outer block's last step: everything to its right, K = the outer block's width
      const int64_t cols_out = n - ob_end_col;
      if (inner_last && cols_out > 0) {
        const int64_t o0 = ob_start * TB, kw = ob_end_col - o0, prow_out = cols_out + m_extra;
        TcSegments so;
        so.nseg = 6;
        for (int q = 0; q < 6; ++q) {
          so.a_k[q] = (int32_t)(kPartA[q] * np + o0);
          so.b_k[q] = (int32_t)(kPartB[q] * np + o0);
        }
        float* Aout = A + ob_end_col * lda + ob_end_col;
        const int64_t wn = cols_out < kNear ? cols_out : kNear;
        TcOperand na{P + ob_end_col * ldp, ldp, true}, nbo{P + ob_end_col * ldp, ldp, true};
        na.kext = nbo.kext = ldp;
        na.mnext = prow_out;
        nbo.mnext = wn;
        sp_status st = gemm_tc(prow_out, wn, kw, -1.f, na, nbo, 1.f, Operand{Aout, SP_F32, lda, 1},
                               OutOperand{Aout, SP_F32, lda}, true, status_dev, sb, &so,
                               (2.0 * (double)prow_out * (double)wn - (double)wn * (double)wn) * (double)kw);
        if (st != SP_OK) return st;
        SP_CUDA_OK(cudaEventRecord(assist->near_done, sb));
        if (cols_out > wn) {
          TcOperand fa{P + (ob_end_col + wn) * ldp, ldp, true}, fb{P + (ob_end_col + wn) * ldp, ldp, true};
          fa.kext = fb.kext = ldp;
          fa.mnext = prow_out - wn;
          fb.mnext = cols_out - wn;
          float* Afar = Aout + wn * lda + wn;
          const double fr = (double)(cols_out - wn);
          st = gemm_tc(prow_out - wn, cols_out - wn, kw, -1.f, fa, fb, 1.f, Operand{Afar, SP_F32, lda, 1},
                       OutOperand{Afar, SP_F32, lda}, true, status_dev, sb, &so,
                       (fr * fr + 2.0 * (double)m_extra * fr) * (double)kw);
          if (st != SP_OK) return st;
        }
      }
    } else if (assist && rem > kNear) {
      // two launches: the first two block columns (all rows below), signalled at once, then the rest
      tb.mnext = kNear;
      sp_status st = gemm_tc(prow, kNear, TB, -1.f, ta, tb, 1.f, Operand{A22, SP_F32, lda, 1},
                             OutOperand{A22, SP_F32, lda}, true, status_dev, sb, &sg,
                             (2.0 * (double)prow * (double)kNear - (double)kNear * (double)kNear) * (double)nb);
      if (st != SP_OK) return st;
      SP_CUDA_OK(cudaEventRecord(assist->near_done, sb));
      TcOperand fa{P + (k0 + nb + kNear) * ldp, ldp, true}, fb{P + (k0 + nb + kNear) * ldp, ldp, true};
      fa.kext = fb.kext = ldp;
      fa.mnext = prow - kNear;
      fb.mnext = rem - kNear;
      float* Afar = A22 + kNear * lda + kNear;
      const double fr = (double)(rem - kNear);
      cudaStream_t sf = sb;
      if (far_apart) {
        sf = assist->far_stream;
        SP_CUDA_OK(cudaStreamWaitEvent(sf, assist->far_go, 0));
      }
      st = gemm_tc(prow - kNear, rem - kNear, TB, -1.f, fa, fb, 1.f, Operand{Afar, SP_F32, lda, 1},
                   OutOperand{Afar, SP_F32, lda}, true, status_dev, sf, &sg,
                   (fr * fr + 2.0 * (double)m_extra * fr) * (double)nb, far_apart ? kFarPairs : 0);
      if (st != SP_OK) return st;
      if (far_apart) {
        SP_CUDA_OK(cudaEventRecord(assist->far_done[kb & 1], sf));
        far_rec[kb & 1] = true;
      }
    } else {
      sp_status st = gemm_tc(prow, rem, TB, -1.f, ta, tb, 1.f, Operand{A22, SP_F32, lda, 1},
                             OutOperand{A22, SP_F32, lda}, true, status_dev, sb, &sg,
                             ((double)rem * (double)rem + 2.0 * (double)m_extra * (double)rem) * (double)nb);
      if (st != SP_OK) return st;
      if (assist) SP_CUDA_OK(cudaEventRecord(assist->near_done, sb));
    }
    if (assist) {
      SP_CUDA_OK(cudaEventRecord(assist->rest_done[kb & 1], sb));
      rec[kb & 1] = true;
    }
  }
  // the factor is complete on `stream` once the assisting stream has drained
  for (int q = 0; q < 2; ++q) {
    if (assist && rec[q]) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->rest_done[q], 0));
    if (far_rec[q]) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->far_done[q], 0));
  }
#undef SP_CUDA_OK
  return SP_OK;
}

sp_status potrs_right_tc(float* X, int64_t m, int64_t n, int64_t ldx, const void* Pv, const float* dinv, void* Xsv,
                         int32_t* status_dev, cudaStream_t stream, const SolveAssist* assist, bool forward_done,
                         const float* Lf, int64_t ldl, int64_t n_factor) {
  const __nv_bfloat16* P = reinterpret_cast<const __nv_bfloat16*>(Pv);
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(Xsv);
  if (n_factor > n && n % TB != 0) return SP_ERR_SHAPE;
  const int64_t np = chol_tc_pad(n_factor > n ? n_factor : n), ldp = 3 * np;
  const int64_t lds = 3 * TB;
  const int64_t nblk = ceil_div(n, (int64_t)TB);
  // Every step applies the inverse diagonal block to one block column (panel) and then updates the columns still to
  // come.  With an assisting stream the update is cut in two: the next block column, which the next panel needs, stays
  // on `stream`; the rest runs on the assisting stream and overlaps the next panel.  Panel jj then needs the "rest"
  // update of step jj - 2 (and reuses its buffer of bf16 parts), which is what the two alternating events order.
#define SP_CUDA_OK(x) do { if ((x) != cudaSuccess) return SP_ERR_CUDA; } while (0)
  // The tensor-core update adds atomically only through its TMA reduction, which needs 16-byte aligned rows of X;
  // without it everything stays on one stream.
  const bool x_al16 = (ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0);
  if (!x_al16) assist = nullptr;
  // Reproducible mode: the far update of a step (assisting stream) and the next step's near update would add into the
  // same columns in an order that depends on timing; on one stream every column receives its updates in step order.
  if (reproducible_mode()) assist = nullptr;
  // Backward sweep: the update of the next block column can ride in the panel kernel (fp32, from the fp32 factor)
  // when the factor's rows are 16-byte aligned too.
  // (its 144 KB of shared memory allow one CTA per SM: only while all row blocks fit in one wave)
  const bool fuse_near = Lf != nullptr && x_al16 && (ldl % 4 == 0) && ((reinterpret_cast<uintptr_t>(Lf) & 15u) == 0) &&
                         ceil_div(m, (int64_t)PA_ROWS) <= 148;
  bool rec[2] = {false, false};
  auto run_sweep = [&](bool forward) -> sp_status {
    for (int64_t step = 0; step < nblk; ++step) {
      const int64_t jb = forward ? step : nblk - 1 - step;
      const int64_t j0 = jb * TB;
      const int nb = (int)((n - j0 < TB) ? (n - j0) : TB);
      const float* dj = dinv + jb * 2 * TB * TB;
      __nv_bfloat16* Xcur = Xs + (step & 1) * m * lds;
      if (assist && rec[step & 1]) SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->rest_done[step & 1], 0));
      // columns still to be updated: [lo, hi)
      const int64_t lo = forward ? j0 + nb : 0, hi = forward ? n : j0;
      // backward: the near columns are the whole block before j (TB wide)
      const bool near_in_panel = !forward && fuse_near && hi > lo;
      PanelNear pn{nullptr, 0, nullptr};
      if (near_in_panel) pn = PanelNear{Lf + j0 * ldl + (hi - TB), ldl, X + (hi - TB)};
      cudaError_t e = forward ? launch_panel_apply<false>(X + j0, ldx, m, nb, dj, Xcur, lds, TB, true, status_dev, stream)
                              : launch_panel_apply<true>(X + j0, ldx, m, nb, dj, Xcur, lds, TB, true, status_dev, stream,
                                                         pn);
      if (e != cudaSuccess) return SP_ERR_CUDA;
      if (hi <= lo) break;
      if (assist) SP_CUDA_OK(cudaEventRecord(assist->panel_done, stream));
      TcOperand ta{Xcur, lds, true};
      ta.kext = lds;
      ta.mnext = m;
      // near part (next block column) and far part of the update
      const int64_t wn = (hi - lo < TB) ? hi - lo : TB;
      const int64_t near_lo = forward ? lo : hi - wn, far_lo = forward ? lo + wn : lo, far_w = hi - lo - wn;
      for (int part = 0; part < 2; ++part) {
        const int64_t c0 = part == 0 ? near_lo : far_lo, w = part == 0 ? wn : far_w;
        if (w <= 0 || (part == 0 && near_in_panel)) continue;
        const bool on_assist = assist && part == 1;
        cudaStream_t st_run = on_assist ? assist->stream : stream;
        if (on_assist) SP_CUDA_OK(cudaStreamWaitEvent(st_run, assist->panel_done, 0));
        TcSegments sg;
        sg.nseg = 6;
        TcOperand tb{nullptr, ldp, forward};
        if (forward) {
          // X[:, c0:c0+w] -= Y_j L[c0:c0+w, j0:j0+nb]^T : B(k, c) = L[c0 + c, j0 + k], K-major rows of P
          tb.ptr = P + c0 * ldp;
          tb.kext = ldp;
          tb.mnext = w;
          for (int q = 0; q < 6; ++q) {
            sg.a_k[q] = kPartA[q] * TB;
            sg.b_k[q] = (int32_t)(kPartB[q] * np + j0);
          }
        } else {
          // X[:, c0:c0+w] -= W_j L[j0:j0+nb, c0:c0+w] : B(k, c) = L[j0 + k, c0 + c], rows of P, columns (N) contiguous
          tb.ptr = P + j0 * ldp;
          tb.kext = n - j0;      // rows of L that exist; beyond them the tensor map returns zero
          tb.mnext = ldp;
          for (int q = 0; q < 6; ++q) {
            sg.a_k[q] = kPartA[q] * TB;
            sg.b_mn[q] = (int32_t)(kPartB[q] * np + c0);
          }
        }
        float* Xc = X + c0;
        sp_status stt = gemm_tc(m, w, TB, -1.f, ta, tb, 1.f, Operand{Xc, SP_F32, ldx, 1}, OutOperand{Xc, SP_F32, ldx},
                                false, status_dev, st_run, &sg, 2.0 * (double)m * (double)w * (double)nb);
        if (stt != SP_OK) return stt;
        if (on_assist) {
          SP_CUDA_OK(cudaEventRecord(assist->rest_done[step & 1], st_run));
          rec[step & 1] = true;
        }
      }
    }
    // the sweep is complete on `stream` once the far updates still in flight have landed
    for (int q = 0; q < 2; ++q)
      if (assist && rec[q]) {
        SP_CUDA_OK(cudaStreamWaitEvent(stream, assist->rest_done[q], 0));
        rec[q] = false;
      }
    return SP_OK;
  };
  if (!forward_done) {               // (done already when X rode along with the factorisation as appended rows)
    sp_status r = run_sweep(true);    // Y L^T = X, block columns left to right
    if (r != SP_OK) return r;
  }
  return run_sweep(false);          // W L = Y, block columns right to left
#undef SP_CUDA_OK
}


// ---------------------------------------------------------------------------------------------------------------
// B independent systems of one size, solved together: every step of the factorisation and of the backward sweep is
// one launch over all systems (diagonal blocks: one CTA per system; panels: grid.y = systems; updates: one batched
// tensor-core launch), so the parallelism comes from the batch and no lookahead or second stream is used.
// Layout: system b at A + b * a_bs ([n + m, n] fp32, the m right-hand sides below the matrix, lda = n), its bf16 parts
// at P + b * (np + m) * 3 np, its inverse diagonal blocks at dinv + b * d_bs, its sweep buffers at Xs + b * 2 m 3 TB.
// n must be a multiple of 128 here (the callers' systems are d x d with d % 128 == 0; others take the plain path).
sp_status potrf_potrs_tc_batched(float* A, int64_t n, int64_t m, int batch, int64_t a_bs, float* dinv, int64_t d_bs,
                                 void* Pv, void* Xsv, int32_t* status_dev, cudaStream_t stream) {
  if (n % TB != 0 || batch < 1 || m < 1) return SP_ERR_SHAPE;
  __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(Pv);
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(Xsv);
  const int64_t np = n, ldp = 3 * np, lda = n;
  const int64_t p_bs = (np + m) * ldp;
  const int64_t nblk = n / TB;
  const int32_t* skip = skip_flag();
  static PerDeviceOnce attr_once;
  if (attr_once.run([] {
        return cudaFuncSetAttribute(chol_diag128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DIAG_SMEM);
      }) != cudaSuccess)
    return SP_ERR_CUDA;
  TcBatch bt;
  bt.nb0 = batch; bt.nb1 = 1;
  bt.a_s0 = bt.b_s0 = p_bs; bt.a_s1 = bt.b_s1 = p_bs;
  bt.c_s0 = bt.cin_s0 = a_bs; bt.c_s1 = bt.cin_s1 = a_bs;
  bt.a_planes = bt.b_planes = 1; bt.a_plane = bt.b_plane = 0;
  // ---- factorisation; the appended rows receive their forward substitution on the way
  for (int64_t kb = 0; kb < nblk; ++kb) {
    const int64_t k0 = kb * TB;
    float* dk = dinv + kb * 2 * TB * TB;
    count_launch();
    chol_diag128_kernel<<<batch, DIAG_THREADS, DIAG_SMEM, stream>>>(A + k0 * lda + k0, lda, TB, dk, k0, status_dev, skip,
                                                                  a_bs, d_bs);
    if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    const int64_t rem = n - k0 - TB, prow = rem + m;
    PanelBatch pb;
    pb.x = a_bs; pb.dinv = d_bs; pb.s = p_bs;
    if (launch_panel_apply<false>(A + (k0 + TB) * lda + k0, lda, prow, TB, dk, P + (k0 + TB) * ldp + k0, ldp, np, true,
                                  status_dev, stream, PanelNear{nullptr, 0, nullptr}, batch, pb) != cudaSuccess)
      return SP_ERR_CUDA;
    if (rem <= 0) break;
    TcOperand ta{P + (k0 + TB) * ldp, ldp, true}, tb{P + (k0 + TB) * ldp, ldp, true};
    ta.kext = tb.kext = ldp;
    ta.mnext = prow;
    tb.mnext = rem;
    TcSegments sg;
    sg.nseg = 6;
    for (int q = 0; q < 6; ++q) {
      sg.a_k[q] = (int32_t)(kPartA[q] * np + k0);
      sg.b_k[q] = (int32_t)(kPartB[q] * np + k0);
    }
    float* A22 = A + (k0 + TB) * lda + (k0 + TB);
    sp_status st = gemm_tc(prow, rem, TB, -1.f, ta, tb, 1.f, Operand{A22, SP_F32, lda, 1}, OutOperand{A22, SP_F32, lda},
                           false, status_dev, stream, &sg,
                           ((double)rem * rem + 2.0 * (double)m * rem) * TB * batch, 0, &bt);
    if (st != SP_OK) return st;
  }
  // ---- backward sweep W L = Y on the appended rows, block columns right to left
  float* X = A + n * lda;                       // [m, n] per system
  const int64_t lds = 3 * TB, xs_bs = 2 * m * lds;
  const bool fuse_near = ceil_div(m, (int64_t)PA_ROWS) * batch <= 148;
  TcBatch bs = bt;
  bs.a_s0 = bs.a_s1 = xs_bs;
  for (int64_t step = 0; step < nblk; ++step) {
    const int64_t jb = nblk - 1 - step, j0 = jb * TB;
    const float* dj = dinv + jb * 2 * TB * TB;
    __nv_bfloat16* Xcur = Xs + (step & 1) * m * lds;
    const bool near_in_panel = fuse_near && j0 > 0;
    PanelNear pn{nullptr, 0, nullptr};
    if (near_in_panel) pn = PanelNear{A + j0 * lda + (j0 - TB), lda, X + (j0 - TB)};
    PanelBatch pb;
    pb.x = a_bs; pb.dinv = d_bs; pb.s = xs_bs; pb.near_l = a_bs;
    if (launch_panel_apply<true>(X + j0, lda, m, TB, dj, Xcur, lds, TB, true, status_dev, stream, pn, batch, pb) !=
        cudaSuccess)
      return SP_ERR_CUDA;
    const int64_t w = near_in_panel ? j0 - TB : j0;     // columns still to be updated by a product: [0, w)
    if (w <= 0) continue;
    TcOperand ta{Xcur, lds, true}, tb{P + j0 * ldp, ldp, false};
    ta.kext = lds;
    ta.mnext = m;
    tb.kext = n - j0;
    tb.mnext = ldp;
    TcSegments sg;
    sg.nseg = 6;
    for (int q = 0; q < 6; ++q) {
      sg.a_k[q] = kPartA[q] * TB;
      sg.b_mn[q] = (int32_t)(kPartB[q] * np);
    }
    sp_status st = gemm_tc(m, w, TB, -1.f, ta, tb, 1.f, Operand{X, SP_F32, lda, 1}, OutOperand{X, SP_F32, lda}, false,
                           status_dev, stream, &sg, 2.0 * (double)m * w * TB * batch, 0, &bs);
    if (st != SP_OK) return st;
  }
  return SP_OK;
}

}  // namespace sp
