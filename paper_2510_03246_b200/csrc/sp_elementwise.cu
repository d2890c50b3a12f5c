// Elementwise and reduction kernels of the ADMM step: the fused auxiliary-variable update (a-update epilogue,
// z^(2), select, dual update, residual and |A| statistics in one pass over the chunk), operand preparation,
// conversions, gathers and small reductions.  All reductions use a fixed order (no floating-point atomics).
#include <algorithm>

#include "sp_common.cuh"

namespace sp {
namespace {

__device__ __forceinline__ float ld_any(const void* p, int32_t dt, int64_t i) {
  return dt == SP_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                       : (dt == SP_F64 ? (float)reinterpret_cast<const double*>(p)[i]
                                       : reinterpret_cast<const float*>(p)[i]);
}

template <typename T>
__device__ __forceinline__ T block_sum(T v, T* smem) {
  // fixed-order tree: warp shuffles, then warp 0 adds the warp results in order
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) smem[w] = v;
  __syncthreads();
  T r = (T)0;
  if (threadIdx.x == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    for (int i = 0; i < nw; ++i) r += smem[i];
  }
  return r;  // valid in thread 0
}

// ------------------------------------------------------------------------------------------------ conversions
__global__ void convert_kernel(const void* src, int32_t sdt, int64_t lds, void* dst, int32_t ddt, int64_t ldd,
                               int64_t rows, int64_t cols) {
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    const int64_t si = i * lds + j, di = i * ldd + j;
    if (sdt == SP_F64) {
      const double v = reinterpret_cast<const double*>(src)[si];
      if (ddt == SP_F64) reinterpret_cast<double*>(dst)[di] = v;
      else if (ddt == SP_BF16) reinterpret_cast<__nv_bfloat16*>(dst)[di] = __float2bfloat16_rn((float)v);
      else reinterpret_cast<float*>(dst)[di] = (float)v;
    } else {
      const float v = ld_any(src, sdt, si);
      if (ddt == SP_F64) reinterpret_cast<double*>(dst)[di] = (double)v;
      else if (ddt == SP_BF16) reinterpret_cast<__nv_bfloat16*>(dst)[di] = __float2bfloat16_rn(v);
      else reinterpret_cast<float*>(dst)[di] = v;
    }
  }
}

// dst[j, i] = src[i, j] through a 32 x 32 shared tile
template <typename TD>
__global__ void transpose_convert_kernel(const float* src, int64_t lds, int64_t rows, int64_t cols, TD* dst,
                                         int64_t ldd) {
  __shared__ float tile[32][33];
  const int64_t c0 = (int64_t)blockIdx.x * 32, r0 = (int64_t)blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int64_t i = r0 + r, j = c0 + threadIdx.x;
    tile[r][threadIdx.x] = (i < rows && j < cols) ? src[i * lds + j] : 0.f;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int64_t j = c0 + r, i = r0 + threadIdx.x;
    if (i < rows && j < cols) {
      if constexpr (sizeof(TD) == 2) dst[j * ldd + i] = __float2bfloat16_rn(tile[threadIdx.x][r]);
      else dst[j * ldd + i] = (TD)tile[threadIdx.x][r];
    }
  }
}

__global__ void split_bf16_kernel(const float* __restrict__ src, int64_t lds, const int32_t* __restrict__ row_idx,
                                  int64_t rows, int64_t cols, int64_t kpad, __nv_bfloat16* __restrict__ dst) {
  const int64_t total = rows * kpad;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / kpad, j = e % kpad;
    __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi;
    if (j < cols) {
      const float v = src[(row_idx ? (int64_t)row_idx[i] : i) * lds + j];
      hi = __float2bfloat16_rn(v);
      lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    dst[i * 2 * kpad + j] = hi;
    dst[i * 2 * kpad + kpad + j] = lo;
  }
}

// dst[i, part * kpad + j] = part `part` of the three-part bf16 split of src[i, j] (hi + mid + lo = src exactly up to
// 2^-24); padding columns are zero.
__global__ void split3_bf16_kernel(const float* __restrict__ src, int64_t lds, int64_t rows, int64_t cols, int64_t kpad,
                                   __nv_bfloat16* __restrict__ dst) {
  const int64_t total = rows * kpad;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / kpad, j = e % kpad;
    const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
    __nv_bfloat16 hi = zero, mid = zero, lo = zero;
    if (j < cols) {
      const float v = src[i * lds + j];
      hi = __float2bfloat16_rn(v);
      const float r1 = v - __bfloat162float(hi);
      mid = __float2bfloat16_rn(r1);
      lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    }
    dst[i * 3 * kpad + j] = hi;
    dst[i * 3 * kpad + kpad + j] = mid;
    dst[i * 3 * kpad + 2 * kpad + j] = lo;
  }
}

__global__ void symmetrize_kernel(float* G, int64_t n, int64_t ld) {
  __shared__ float tile[32][33];
  // block (bx, by) with bx > by mirrors lower tile (row block bx, col block by) to (by, bx); diagonal blocks in place
  const int64_t bx = blockIdx.x, by = blockIdx.y;
  if (bx < by) return;
  const int64_t r0 = bx * 32, c0 = by * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int64_t i = r0 + r, j = c0 + threadIdx.x;
    tile[r][threadIdx.x] = (i < n && j < n) ? G[i * ld + j] : 0.f;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int64_t i = c0 + r, j = r0 + threadIdx.x;  // element (i, j) of the upper part = lower (j, i)
    if (i < n && j < n && j > i) G[i * ld + j] = tile[threadIdx.x][r];
  }
}

template <typename T>
__global__ void load_spd_kernel(const float* G, int64_t ldg, const int32_t* idx, int64_t n, const double* rho, T* dst,
                                int64_t ldd, const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;   // conditional launch (see SkipScope)
  const double r = rho ? rho[0] : 0.0;
  const int64_t total = n * n;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / n, j = e % n;
    if (j > i) continue;
    const int64_t gi = idx ? idx[i] : i, gj = idx ? idx[j] : j;
    // the lower triangle of G is authoritative: read (max, min)
    const int64_t a = gi > gj ? gi : gj, b = gi > gj ? gj : gi;
    double v = (double)G[a * ldg + b];
    if (i == j) v += r;
    dst[i * ldd + j] = (T)v;
  }
}

template <typename T>
__global__ void gather_cols_kernel(const float* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k, T* dst,
                                   int64_t ldd, const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  const int64_t total = rows * k;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / k, a = e % k;
    dst[i * ldd + a] = (T)src[i * lds + (idx ? idx[a] : a)];
  }
}

__global__ void gather_rows_kernel(const float* __restrict__ src, int64_t lds, const int32_t* __restrict__ idx,
                                   int64_t rows, int64_t cols, float* __restrict__ dst, int64_t ldd) {
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    dst[i * ldd + j] = src[(int64_t)idx[i] * lds + j];
  }
}

template <typename T>
__global__ void scatter_cols_kernel(const T* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k,
                                    float* dst, int64_t ldd, const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  const int64_t total = rows * k;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / k, a = e % k;
    dst[i * ldd + (idx ? idx[a] : a)] = (float)src[i * lds + a];
  }
}

__global__ void fill_zero_kernel(float* dst, int64_t ld, int64_t rows, int64_t cols, const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x)
    dst[(e / cols) * ld + (e % cols)] = 0.f;
}

// dst[i, 0:kpad] = src[i, 0:k] followed by zeros
__global__ void copy_cols_padded_kernel(const float* __restrict__ src, int64_t lds, int64_t rows, int64_t k,
                                        int64_t kpad, float* __restrict__ dst) {
  const int64_t total = rows * kpad;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / kpad, a = e % kpad;
    dst[e] = a < k ? src[i * lds + a] : 0.f;
  }
}

__global__ void effective_ridge_kernel(const float* G, int64_t ldg, int64_t n, double rho, int rel, double* out) {
  __shared__ double sm[32];
  double s = 0.0;
  if (rel)
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) s += (double)G[i * ldg + i];
  s = block_sum<double>(s, sm);
  if (threadIdx.x == 0) out[0] = rel ? rho * s / (double)n : rho;
}

// ------------------------------------------------------------------------------------------------ chunk kernels
// The kept units of a module are a subset S of its n channels.  Tensors that exist only on S are stored COMPACT:
// column p of a compact [T, k] tensor belongs to channel idx[p] (idx ascending).  For the elementwise kernels the
// channels are cut into groups of 8 consecutive ones: grp_base[g] = number of kept channels before channel 8 g,
// grp_mask[g] = bit q set when channel 8 g + q is kept.  The kept channels of a group then sit at compact positions
// grp_base[g], grp_base[g] + 1, ... in channel order.
__global__ void __launch_bounds__(1024) group_map_kernel(const uint8_t* __restrict__ mask, int64_t n,
                                                         int32_t* grp_base, uint8_t* grp_mask) {
  __shared__ int warp_tot[32];
  __shared__ int s_before;
  const int64_t groups = ceil_div(n, (int64_t)8);
  if (threadIdx.x == 0) s_before = 0;
  __syncthreads();
  for (int64_t g0 = 0; g0 < groups; g0 += blockDim.x) {
    const int64_t g = g0 + threadIdx.x;
    unsigned bits = 0;
    if (g < groups)
      for (int q = 0; q < 8; ++q)
        if (8 * g + q < n && mask[8 * g + q]) bits |= 1u << q;
    const int cnt = __popc(bits);
    // inclusive scan of cnt over the block
    int v = cnt;
    const int l = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (l >= o) v += u;
    }
    if (l == 31) warp_tot[w] = v;
    __syncthreads();
    int before = s_before;
    for (int i = 0; i < w; ++i) before += warp_tot[i];
    if (g < groups) {
      grp_base[g] = before + v - cnt;
      grp_mask[g] = (uint8_t)bits;
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) s_before = before + v;
    __syncthreads();
  }
}

__device__ __forceinline__ void store8(void* base, int32_t dt, int64_t e, const float* v) {
  if (dt == SP_BF16) {
    __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 h2 = __floats2bfloat162_rn(v[4], v[5]), h3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&h0); pk.y = *reinterpret_cast<uint32_t*>(&h1);
    pk.z = *reinterpret_cast<uint32_t*>(&h2); pk.w = *reinterpret_cast<uint32_t*>(&h3);
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(base) + e) = pk;
  } else {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + e) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + e + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// H_S = storage(phi(Z) - U) on the kept channels, compact [T, ldh].  A thread owns 8 consecutive COMPACT columns: it
// gathers their channels (ascending, so close together in a row of Z) and writes one 16-byte (bf16) or two 16-byte
// (fp32) vectors per row.  Columns k..ldh-1 of H are written as zero.
// lo_off > 0 (bf16 only): H holds two parts side by side, bf16(h) in columns [0, ncols) and bf16(h - bf16(h)) in columns
// [lo_off, lo_off + ncols), so that a product with H keeps about 16 bits of h (two K segments of the GEMM).
__global__ void __launch_bounds__(256) prep_h_kernel(const float* __restrict__ Z, const float* __restrict__ U,
                                                     const float* __restrict__ G, void* __restrict__ H, int32_t hdt,
                                                     int64_t T, int64_t n,
                                                     int64_t ldh, int64_t ncols, int64_t lo_off, int64_t k,
                                                     const int32_t* __restrict__ idx, int32_t rows_per_block,
                                                     const int32_t* skip) {
  if (skip != nullptr && *skip != 0) return;   // conditional launch (see SkipScope)
  const int64_t p0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (p0 >= ncols) return;
  int ch[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) ch[q] = (p0 + q < k) ? idx[p0 + q] : -1;
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per_block;
  const int64_t r_end = (r_begin + rows_per_block < T) ? r_begin + rows_per_block : T;
#pragma unroll 2
  for (int64_t r = r_begin; r < r_end; ++r) {
    const float* zr = Z + r * n;
    float h[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) h[q] = (ch[q] >= 0) ? (G ? zr[ch[q]] : fmaxf(zr[ch[q]], 0.f)) : 0.f;
    if (G) {           // gated module: phi(z) = g z
      const float* gr = G + r * n;
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (ch[q] >= 0) h[q] *= gr[ch[q]];
    }
    if (U) {
      const float* ur = U + r * n;
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (ch[q] >= 0) h[q] -= ur[ch[q]];
    }
    store8(H, hdt, r * ldh + p0, h);
    if (lo_off > 0) {
#pragma unroll
      for (int q = 0; q < 8; ++q) h[q] -= __bfloat162float(__float2bfloat16_rn(h[q]));
      store8(H, hdt, r * ldh + lo_off + p0, h);
    }
  }
}

// One element of the fused update.  Returns A; writes the new z (and u).
constexpr int kZGated = 2;   // internal rule of gated modules: phi(z) = gate * z, one closed-form minimiser

__device__ __forceinline__ float update_one(float zold, float z1, float dcorr, float& u, bool has_u, float alpha,
                                            float beta, float inv_ab, int z_rule, float gate, float& znew) {
  if (z_rule == kZGated) {
    const float h = gate * zold - (has_u ? u : 0.f);
    const float a = h + dcorr;
    const float au = a + (has_u ? u : 0.f);
    // The divisor lies in [alpha, alpha + beta g^2], far from the ends of the exponent range, so its correctly
    // rounded reciprocal never leaves the fast path.  A plain division also inspects the numerator, which is tiny
    // wherever the gate factor is: with wide-ranged gate inputs its out-of-range path made the kernel 45 % slower.
    znew = (beta * gate * au + alpha * z1) * __frcp_rn(fmaf(beta * gate, gate, alpha));
    if (has_u) u = u + a - gate * znew;
    return a;
  }
  const float h = fmaxf(zold, 0.f) - (has_u ? u : 0.f);
  const float a = h + dcorr;
  const float au = a + (has_u ? u : 0.f);
  const float z2 = (beta * au + alpha * z1) * inv_ab;
  if (z_rule == SP_Z_PAPER) {
    znew = (zold < 0.f) ? z1 : z2;
  } else {
    const float zn = fminf(z1, 0.f), zp = fmaxf(z2, 0.f);
    const float fn = beta * au * au + alpha * (zn - z1) * (zn - z1);
    const float fp = beta * (au - zp) * (au - zp) + alpha * (zp - z1) * (zp - z1);
    znew = (fn < fp) ? zn : zp;
  }
  if (has_u) u = u + a - fmaxf(znew, 0.f);
  return a;
}

__device__ __forceinline__ void store4(void* base, int32_t dt, int64_t e, const float* v) {
  if (dt == SP_BF16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(base) + e) = pk;
  } else {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + e) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

// The fused auxiliary-variable update of one chunk: per element a = h + D (h = phi(z) - u), z2, the select, the dual
// update, the residual / norm partial sums and the column sums of |a|, reading Z (and U) once and writing Z (and U),
// A and the storage copy of Z once.  D and z1 exist on the kept channels only (compact, see above); on a pruned
// channel both are zero (its row of W1 and its row of Q are zero).
// grid: (column blocks of 1024 channels, row blocks).  A thread owns 4 consecutive channels and walks its rows two at
// a time: all loads of both rows are issued before the first store, so that enough bytes are in flight per SM to
// cover the DRAM latency (the kernel moves 12 n + 8 k bytes per token and does almost no arithmetic).
// Sums: fp32 within one row and per column over the thread's rows (at most a few hundred terms), fp64 across rows
// and blocks.
// Transposed-A tile of one block: kAtRows rows (64-byte pieces per channel) of its 1024 channels, channel-major with a
// pitch of 72 bytes.  (A layout free of bank conflicts, written out in 8-byte pieces, measured 2 % slower: the kernel
// is bound by its global stores, not by shared memory.)
constexpr int kAtRows = 32;
constexpr int kAtPitch = kAtRows + 4;                 // bf16 elements
constexpr size_t kAtTileBytes = (size_t)1024 * kAtPitch * sizeof(__nv_bfloat16);

template <bool HAS_U>
struct UpdRow {
  float zo[4], u[4], z1[4], dc[4], gt[4];
};

template <bool HAS_U, int Z_RULE>
__global__ void __launch_bounds__(256, 2) fused_update_kernel(UpdateArgs g) {
  __shared__ double sm[32];
  const int64_t grp4 = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t c0 = grp4 * 4;
  int64_t rows_per = ceil_div(g.T, (int64_t)g.row_blocks);
  if (g.At_out) rows_per = (rows_per + kAtRows - 1) / kAtRows * kAtRows;   // whole tiles: 16-byte aligned pieces
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per;
  const int64_t r_end = (r_begin + rows_per < g.T) ? r_begin + rows_per : g.T;
  const float inv_ab = 1.f / (g.alpha + g.beta);
  float* __restrict__ Zp = g.Z;
  float* __restrict__ Up = g.U;
  const float* __restrict__ z1p = g.z1;
  const float* __restrict__ Dp = g.D;
  double s_res = 0.0, s_z = 0.0, s_a = 0.0, s_in = 0.0;
  float cs[4] = {0.f, 0.f, 0.f, 0.f};
  // With a transposed A every warp stages kAtRows rows of its 128 channels in shared memory (channel-major) and
  // writes them out as 64-byte pieces; lanes beyond the last channel walk the loop too (without touching memory),
  // so that the warp-level barriers see all lanes.
  extern __shared__ __align__(16) __nv_bfloat16 at_tile[];     // [1024][kAtPitch], only with At_out
  __shared__ int32_t at_row[1024];                             // row of each channel of the block in "kept first" order
  const bool active = c0 < g.n;
  {
    const int cnt = !active ? 0 : (g.n - c0 >= 4) ? 4 : (int)(g.n - c0);
    const bool vec = (g.n % 4 == 0);
    // kept channels of this half group and their compact offsets
    const unsigned bits8 = active ? g.grp_mask[grp4 >> 1] : 0u;
    const bool upper = (grp4 & 1) != 0;
    const unsigned bits = upper ? (bits8 >> 4) : (bits8 & 0xFu);
    const int base = active ? g.grp_base[grp4 >> 1] + (upper ? __popc(bits8 & 0xFu) : 0) : 0;
    int off[4];
    {
      int pos = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        off[q] = pos;
        pos += (bits >> q) & 1u;
      }
    }
    if (g.at_kept_first) {
      // looked up once: kept channel -> its compact position, pruned channel -> k + its rank among the pruned ones
      // (only the warp that owns the channels reads them back: a warp-level barrier below is enough)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int kb = base + off[q];
        at_row[4 * (int)threadIdx.x + q] = ((bits >> q) & 1u) ? kb : (int32_t)(g.k + (c0 + q - kb));
      }
      __syncwarp();
    }
    auto load_row = [&](int64_t r, UpdRow<HAS_U>& w) {
      const int64_t e = r * g.n + c0;
      if (vec) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(Zp + e));     // read once: streaming
        w.zo[0] = v.x; w.zo[1] = v.y; w.zo[2] = v.z; w.zo[3] = v.w;
        if (HAS_U) {
          const float4 x = *reinterpret_cast<const float4*>(Up + e);
          w.u[0] = x.x; w.u[1] = x.y; w.u[2] = x.z; w.u[3] = x.w;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          w.zo[q] = (q < cnt) ? Zp[e + q] : 0.f;
          if (HAS_U) w.u[q] = (q < cnt) ? Up[e + q] : 0.f;
        }
      }
      if (!HAS_U) {
#pragma unroll
        for (int q = 0; q < 4; ++q) w.u[q] = 0.f;
      }
      if (Z_RULE == kZGated) {
        if (vec) {
          const float4 x = *reinterpret_cast<const float4*>(g.gate + e);
          w.gt[0] = x.x; w.gt[1] = x.y; w.gt[2] = x.z; w.gt[3] = x.w;
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q) w.gt[q] = (q < cnt) ? g.gate[e + q] : 0.f;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) w.gt[q] = 0.f;
      }
      const float* zp = z1p + r * g.ldk + base;
      const float* dp = Dp + r * g.ldk + base;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool kept = (bits >> q) & 1u;
        // (plain loads: a warp's run of kept channels starts and ends inside sectors that the neighbouring warps read too)
        w.z1[q] = kept ? zp[off[q]] : 0.f;
        w.dc[q] = kept ? dp[off[q]] : 0.f;
      }
    };
    auto finish_row = [&](int64_t r, UpdRow<HAS_U>& w, __nv_bfloat16* arow) {
      const int64_t e = r * g.n + c0;
      float a[4], zn[4];
      float p_res = 0.f, p_z = 0.f, p_a = 0.f, p_in = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        a[q] = update_one(w.zo[q], w.z1[q], w.dc[q], w.u[q], HAS_U, g.alpha, g.beta, inv_ab, Z_RULE, w.gt[q], zn[q]);
        if (!vec && q >= cnt) { a[q] = 0.f; zn[q] = 0.f; w.z1[q] = 0.f; }
        const float din = zn[q] - w.z1[q];
        p_in = fmaf(din, din, p_in);
        const float diff = a[q] - (Z_RULE == kZGated ? w.gt[q] * zn[q] : fmaxf(zn[q], 0.f));
        p_res = fmaf(diff, diff, p_res);
        p_z = fmaf(zn[q], zn[q], p_z);
        p_a = fmaf(a[q], a[q], p_a);
        cs[q] += fabsf(a[q]);
      }
      s_res += (double)p_res;
      s_z += (double)p_z;
      s_a += (double)p_a;
      s_in += (double)p_in;
      if (vec) {
        // Z and its operands are touched once per step: streaming accesses keep them from displacing the transposed A,
        // which the accumulator products read next (measured: 6.8 against 6.95 ms per C2 step)
        __stcs(reinterpret_cast<float4*>(Zp + e), make_float4(zn[0], zn[1], zn[2], zn[3]));
        if (HAS_U) *reinterpret_cast<float4*>(Up + e) = make_float4(w.u[0], w.u[1], w.u[2], w.u[3]);
        if (g.At_out) {
#pragma unroll
          for (int q = 0; q < 4; ++q) arow[q] = __float2bfloat16_rn(a[q]);
        } else {
          store4(g.A_out, g.out_dtype, e, a);
        }
        if (g.Zb_out) store4(g.Zb_out, g.out_dtype, e, zn);
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (q < cnt) {
            Zp[e + q] = zn[q];
            if (HAS_U) Up[e + q] = w.u[q];
            if (g.out_dtype == SP_BF16) {
              reinterpret_cast<__nv_bfloat16*>(g.A_out)[e + q] = __float2bfloat16_rn(a[q]);
              if (g.Zb_out) reinterpret_cast<__nv_bfloat16*>(g.Zb_out)[e + q] = __float2bfloat16_rn(zn[q]);
            } else {
              reinterpret_cast<float*>(g.A_out)[e + q] = a[q];
              if (g.Zb_out) reinterpret_cast<float*>(g.Zb_out)[e + q] = zn[q];
            }
          }
        }
      }
    };
    const int ct = 4 * (int)threadIdx.x;                    // first of this thread's channels inside the block
    const int64_t tile_step = g.At_out ? kAtRows : (r_end > r_begin ? r_end - r_begin : 1);
    for (int64_t rt = r_begin; rt < r_end; rt += tile_step) {
      const int64_t rt_end = (rt + tile_step < r_end) ? rt + tile_step : r_end;
      if (active) {
        int64_t r = rt;
        for (; r + 3 < rt_end; r += 4) {
          UpdRow<HAS_U> w0, w1, w2, w3;
          load_row(r, w0);
          load_row(r + 1, w1);
          load_row(r + 2, w2);
          load_row(r + 3, w3);
          __align__(8) __nv_bfloat16 ab[4][4];
          finish_row(r, w0, ab[0]);
          finish_row(r + 1, w1, ab[1]);
          finish_row(r + 2, w2, ab[2]);
          finish_row(r + 3, w3, ab[3]);
          if (g.At_out) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              __align__(8) __nv_bfloat16 col[4] = {ab[0][q], ab[1][q], ab[2][q], ab[3][q]};
              *reinterpret_cast<uint2*>(&at_tile[(ct + q) * kAtPitch + (int)(r - rt)]) =
                  *reinterpret_cast<const uint2*>(col);
            }
          }
        }
        for (; r < rt_end; ++r) {
          UpdRow<HAS_U> w0;
          __nv_bfloat16 ab1[4];
          load_row(r, w0);
          finish_row(r, w0, ab1);
          if (g.At_out) {
#pragma unroll
            for (int q = 0; q < 4; ++q) at_tile[(ct + q) * kAtPitch + (int)(r - rt)] = ab1[q];
          }
        }
      }
      if (g.At_out) {
        // write the tile out, each warp its own 128 channels (only the warp itself wrote them, so a warp-level
        // barrier is enough): rows rt .. rt_end - 1 of a channel in pieces of 8 rows (16 bytes), 4 lanes per channel
        __syncwarp();
        const int rows_here = (int)(rt_end - rt);
        const int lane = (int)threadIdx.x & 31, wch0 = ((int)threadIdx.x >> 5) * 128;
        const int64_t cb = (int64_t)blockIdx.x * 1024 + wch0;
        const int nch = (g.n - cb < 128) ? (int)((g.n - cb > 0) ? g.n - cb : 0) : 128;
        __nv_bfloat16* At = reinterpret_cast<__nv_bfloat16*>(g.At_out);
        for (int e = lane; e < nch * (kAtRows / 8); e += 32) {
          const int ch = e / (kAtRows / 8), piece = e % (kAtRows / 8);
          const __nv_bfloat16* src = &at_tile[(wch0 + ch) * kAtPitch + piece * 8];
          const int64_t row = g.at_kept_first ? (int64_t)at_row[(wch0 + ch)] : cb + ch;
          __nv_bfloat16* dst = At + row * g.ldt + rt + piece * 8;
          if (piece * 8 + 8 <= rows_here) {
            const uint2 lo = *reinterpret_cast<const uint2*>(src), hi = *reinterpret_cast<const uint2*>(src + 4);
            *reinterpret_cast<uint4*>(dst) = make_uint4(lo.x, lo.y, hi.x, hi.y);
          } else {
            for (int q = 0; q < 8; ++q)
              if (piece * 8 + q < rows_here) dst[q] = src[q];
          }
        }
        __syncwarp();
      }
    }
    if (g.absA_part && active) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (q < cnt) g.absA_part[(int64_t)blockIdx.y * g.n + c0 + q] = (double)cs[q];
    }
  }
  const int64_t bid = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
  const double r0 = block_sum<double>(s_res, sm);
  const double r1 = block_sum<double>(s_z, sm);
  const double r2 = block_sum<double>(s_a, sm);
  const double r3 = block_sum<double>(s_in, sm);
  if (threadIdx.x == 0) {
    g.partial[bid * 4 + 0] = r0;
    g.partial[bid * 4 + 1] = r1;
    g.partial[bid * 4 + 2] = r2;
    g.partial[bid * 4 + 3] = r3;
  }
}

// The fused update of a chunk in the form that also leaves what the NEXT step reads (bf16 storage, ReLU, no dual
// variable, n % 4 == 0, accumulators kept in "kept channels first" order).  Besides the new Z (fp32, in place) and the
// transposed A it writes, from the same registers,
//   Zt[row(c), t] = bf16(Z_new[t, c])          the K-major operand of R1 = Z^T X: the kept channels' rows always, the
//                                              pruned ones only when *zt_pruned_flag != 0 (their part of R1 is a scaled
//                                              copy of the step before while the mask stays),
//   Ht[p(c), t]   = bf16(max(Z_new[t, c], 0))  for the kept channels: h of the next step's a-update, transposed,
// so that Z is read once and written once per step and no separate pass over the new Z is needed.
// A warp owns 64 channels (a thread 2 consecutive ones) and 32 rows at a time: four rounds of eight rows, all loads
// of a round in flight before its first store.  The warp stages its rows of a and z_new in two shared tiles of its own
// (channel-major) and writes the 32 rows of every channel out as 64-byte pieces.  A block owns 128 channels: four of
// its warps own the same 64 and take the row tiles in turn, so that the four 64-byte pieces of 256 consecutive bytes
// of an output row are written at about the same time (no barrier: the warps only happen to run side by side) and
// leave the L2 as whole lines — 6.6 against 7.3 ms per C2 step with every warp on channels of its own.  (A form in
// which two warps shared 128 channels and met at a barrier before the write-out, and one in which each of them wrote
// 32-byte pieces, measured 13 % and 6 % slower than the latter.)
constexpr int kNextTiles = 4;            // warps that own the same 64 channels and take row tiles in turn
constexpr int kNextChannels = 512 / kNextTiles;       // channels of a block
constexpr size_t kNextTileBytes = (size_t)2 * 512 * kAtPitch * sizeof(__nv_bfloat16);

__device__ __forceinline__ uint32_t relu_bf16x2(uint32_t v) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&v);
  x = __hmax2(x, __float2bfloat162_rn(0.f));
  return *reinterpret_cast<uint32_t*>(&x);
}

struct NextRow {
  float zo[2], z1[2], dc[2];
};

template <int Z_RULE>
__global__ void __launch_bounds__(256, 2) fused_update_next_kernel(UpdateArgs g) {
  __shared__ double sm[32];
  extern __shared__ __align__(16) __nv_bfloat16 next_tiles[];  // a_tile[512][kAtPitch], then z_tile[512][kAtPitch]
  __shared__ int32_t at_row[512];                              // per warp: row of each of its channels in "kept first" order
  __nv_bfloat16* a_tile = next_tiles;
  __nv_bfloat16* z_tile = next_tiles + 512 * kAtPitch;
  const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5;
  const int hw = warp / (8 / kNextTiles);                       // which of the interleaved row tiles
  const int64_t cb = (int64_t)blockIdx.x * kNextChannels + (warp % (8 / kNextTiles)) * 64;      // the warp's 64 channels
  const int64_t c0 = cb + 2 * lane;
  int64_t rows_per = ceil_div(g.T, (int64_t)g.row_blocks);
  rows_per = (rows_per + kNextTiles * kAtRows - 1) / (kNextTiles * kAtRows) * (kNextTiles * kAtRows);
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per;
  const int64_t r_end = (r_begin + rows_per < g.T) ? r_begin + rows_per : g.T;
  const float inv_ab = 1.f / (g.alpha + g.beta);
  float* __restrict__ Zp = g.Z;
  const float* __restrict__ z1p = g.z1;
  const float* __restrict__ Dp = g.D;
  double s_res = 0.0, s_z = 0.0, s_a = 0.0, s_in = 0.0;
  float cs[2] = {0.f, 0.f};
  const bool active = c0 < g.n;                                 // n % 4 == 0: a thread's channels exist together
  const unsigned bits8 = active ? g.grp_mask[c0 >> 3] : 0u;
  const int sh = (int)(c0 & 7);                                 // 0, 2, 4, 6
  const unsigned bits = (bits8 >> sh) & 3u;
  const int base = active ? g.grp_base[c0 >> 3] + __popc(bits8 & ((1u << sh) - 1u)) : 0;
  const int off1 = (int)(bits & 1u);
  const int ct = warp * 64 + 2 * lane;                          // first of this thread's channels inside the block
  {
    // (only the warp itself reads its entries back: a warp-level barrier is enough)
    at_row[ct] = (bits & 1u) ? base : (int32_t)(g.k + (c0 - base));
    at_row[ct + 1] = (bits & 2u) ? base + off1 : (int32_t)(g.k + (c0 + 1 - (base + off1)));
    __syncwarp();
  }
  const bool write_pruned_z = g.zt_pruned_flag == nullptr || *g.zt_pruned_flag != 0;
  auto load_row = [&](int64_t r, NextRow& w) {
    const float2 v = __ldcs(reinterpret_cast<const float2*>(Zp + r * g.n + c0));     // read once: streaming
    w.zo[0] = v.x; w.zo[1] = v.y;
    const float* zp = z1p + r * g.ldk + base;
    const float* dp = Dp + r * g.ldk + base;
    // (plain loads: a warp's run of kept channels starts and ends inside sectors that the neighbouring warps read too)
    w.z1[0] = (bits & 1u) ? zp[0] : 0.f;
    w.dc[0] = (bits & 1u) ? dp[0] : 0.f;
    w.z1[1] = (bits & 2u) ? zp[off1] : 0.f;
    w.dc[1] = (bits & 2u) ? dp[off1] : 0.f;
  };
  auto finish_row = [&](int64_t r, NextRow& w, __nv_bfloat16& a0, __nv_bfloat16& a1, __nv_bfloat16& zb0,
                        __nv_bfloat16& zb1) {
    float a[2], zn[2];
    float p_res = 0.f, p_z = 0.f, p_a = 0.f, p_in = 0.f;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      float u = 0.f;
      a[q] = update_one(w.zo[q], w.z1[q], w.dc[q], u, false, g.alpha, g.beta, inv_ab, Z_RULE, 0.f, zn[q]);
      const float din = zn[q] - w.z1[q];
      p_in = fmaf(din, din, p_in);
      const float diff = a[q] - fmaxf(zn[q], 0.f);
      p_res = fmaf(diff, diff, p_res);
      p_z = fmaf(zn[q], zn[q], p_z);
      p_a = fmaf(a[q], a[q], p_a);
      cs[q] += fabsf(a[q]);
    }
    a0 = __float2bfloat16_rn(a[0]); a1 = __float2bfloat16_rn(a[1]);
    zb0 = __float2bfloat16_rn(zn[0]); zb1 = __float2bfloat16_rn(zn[1]);
    s_res += (double)p_res;
    s_z += (double)p_z;
    s_a += (double)p_a;
    s_in += (double)p_in;
    __stcs(reinterpret_cast<float2*>(Zp + r * g.n + c0), make_float2(zn[0], zn[1]));
  };
  __nv_bfloat16* At = reinterpret_cast<__nv_bfloat16*>(g.At_out);
  __nv_bfloat16* Zt = reinterpret_cast<__nv_bfloat16*>(g.Zt_out);
  __nv_bfloat16* Ht = reinterpret_cast<__nv_bfloat16*>(g.Ht_out);
  const int nch = (g.n - cb < 64) ? (int)((g.n - cb > 0) ? g.n - cb : 0) : 64;
  for (int64_t rt = r_begin + hw * kAtRows; rt < r_end; rt += kNextTiles * kAtRows) {
    const int64_t rt_end = (rt + kAtRows < r_end) ? rt + kAtRows : r_end;
    if (active) {
      int64_t r = rt;
      for (; r + 7 < rt_end; r += 8) {
        NextRow w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) load_row(r + i, w[i]);
        __align__(16) __nv_bfloat16 ca[2][8], cz[2][8];
#pragma unroll
        for (int i = 0; i < 8; ++i) finish_row(r + i, w[i], ca[0][i], ca[1][i], cz[0][i], cz[1][i]);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          // (kAtPitch = 36 elements: a row of the tile starts 8-byte aligned, so two 8-byte stores)
          const int at = (ct + q) * kAtPitch + (int)(r - rt);
          uint2* da = reinterpret_cast<uint2*>(&a_tile[at]);
          uint2* dz = reinterpret_cast<uint2*>(&z_tile[at]);
          da[0] = *reinterpret_cast<const uint2*>(&ca[q][0]);
          da[1] = *reinterpret_cast<const uint2*>(&ca[q][4]);
          dz[0] = *reinterpret_cast<const uint2*>(&cz[q][0]);
          dz[1] = *reinterpret_cast<const uint2*>(&cz[q][4]);
        }
      }
      for (; r < rt_end; ++r) {
        NextRow w0;
        __nv_bfloat16 a0, a1, zb0, zb1;
        load_row(r, w0);
        finish_row(r, w0, a0, a1, zb0, zb1);
        const int at = ct * kAtPitch + (int)(r - rt);
        a_tile[at] = a0; a_tile[at + kAtPitch] = a1;
        z_tile[at] = zb0; z_tile[at + kAtPitch] = zb1;
      }
    }
    __syncwarp();
    // the warp writes its 64 channels out: rows rt .. rt_end - 1 of a channel in pieces of 8 rows (16 bytes), 4 lanes
    // per channel
    const int rows_here = (int)(rt_end - rt);
    for (int e = lane; e < nch * (kAtRows / 8); e += 32) {
      const int ch = e / (kAtRows / 8), piece = e % (kAtRows / 8);
      const int at = (warp * 64 + ch) * kAtPitch + piece * 8;
      const int64_t row = at_row[warp * 64 + ch];
      const bool kept = row < g.k;
      const int64_t dst = row * g.ldt + rt + piece * 8;
      if (piece * 8 + 8 <= rows_here) {
        const uint2 alo = *reinterpret_cast<const uint2*>(&a_tile[at]), ahi = *reinterpret_cast<const uint2*>(&a_tile[at + 4]);
        *reinterpret_cast<uint4*>(At + dst) = make_uint4(alo.x, alo.y, ahi.x, ahi.y);
        if (kept || write_pruned_z) {
          const uint2 zlo = *reinterpret_cast<const uint2*>(&z_tile[at]), zhi = *reinterpret_cast<const uint2*>(&z_tile[at + 4]);
          *reinterpret_cast<uint4*>(Zt + dst) = make_uint4(zlo.x, zlo.y, zhi.x, zhi.y);
          if (kept)
            *reinterpret_cast<uint4*>(Ht + dst) =
                make_uint4(relu_bf16x2(zlo.x), relu_bf16x2(zlo.y), relu_bf16x2(zhi.x), relu_bf16x2(zhi.y));
        }
      } else {
        const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
        for (int q = 0; q < 8; ++q)
          if (piece * 8 + q < rows_here) {
            At[dst + q] = a_tile[at + q];
            if (kept || write_pruned_z) Zt[dst + q] = z_tile[at + q];
            if (kept) Ht[dst + q] = __hgt(z_tile[at + q], zero) ? z_tile[at + q] : zero;
          }
      }
    }
    __syncwarp();
  }
  if (active && g.absA_part) {
    // (kNextTiles warps per channel: the partial sums have kNextTiles * row_blocks rows)
    g.absA_part[((int64_t)blockIdx.y * kNextTiles + hw) * g.n + c0] = (double)cs[0];
    g.absA_part[((int64_t)blockIdx.y * kNextTiles + hw) * g.n + c0 + 1] = (double)cs[1];
  }
  const int64_t bid = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;
  const double r0 = block_sum<double>(s_res, sm);
  const double r1 = block_sum<double>(s_z, sm);
  const double r2 = block_sum<double>(s_a, sm);
  const double r3 = block_sum<double>(s_in, sm);
  if (threadIdx.x == 0) {
    g.partial[bid * 4 + 0] = r0;
    g.partial[bid * 4 + 1] = r1;
    g.partial[bid * 4 + 2] = r2;
    g.partial[bid * 4 + 3] = r3;
  }
}

// h of a step whose mask differs from the one the last token pass left h for (bf16 storage, ReLU, no dual variable,
// n % 4 == 0): Ht[p(c), t] = bf16(max(Z[t, c], 0)) for the kept channels c, p(c) = its rank among them — the transposed
// layout in which the fused update above leaves it.  A thread owns 4 consecutive channels, a warp stages kAtRows rows
// of its 128 channels in shared memory and writes the kept ones out as 64-byte pieces.
__global__ void __launch_bounds__(256, 3) gather_ht_kernel(const float* __restrict__ Z, int64_t T, int64_t n, int64_t k,
                                                           const int32_t* __restrict__ grp_base,
                                                           const uint8_t* __restrict__ grp_mask,
                                                           __nv_bfloat16* __restrict__ Ht, int64_t ldt,
                                                           int32_t row_blocks, const int32_t* __restrict__ skip) {
  if (skip != nullptr && *skip != 0) return;
  extern __shared__ __align__(16) __nv_bfloat16 zt_tile[];     // [1024][kAtPitch]
  __shared__ int32_t row_of[8][128];                           // per warp: row of each of its channels in Ht, -1: pruned
  const int64_t grp4 = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t c0 = grp4 * 4;
  int64_t rows_per = ceil_div(T, (int64_t)row_blocks);
  rows_per = (rows_per + kAtRows - 1) / kAtRows * kAtRows;
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per;
  const int64_t r_end = (r_begin + rows_per < T) ? r_begin + rows_per : T;
  const bool active = c0 < n;                                   // n % 4 == 0: a thread's channels exist together
  const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5;
  const unsigned bits8 = active ? grp_mask[grp4 >> 1] : 0u;
  const bool upper = (grp4 & 1) != 0;
  const unsigned bits = upper ? (bits8 >> 4) : (bits8 & 0xFu);
  const int base = active ? grp_base[grp4 >> 1] + (upper ? __popc(bits8 & 0xFu) : 0) : 0;
  {
    int kb = base;       // kept channels before channel c0 + q
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const bool is_kept = (bits >> q) & 1u;
      // (a mask that keeps more channels than k is reported elsewhere; its surplus channels are not written)
      row_of[warp][4 * lane + q] = (is_kept && kb < k) ? kb : -1;
      kb += is_kept ? 1 : 0;
    }
  }
  __syncwarp();
  const int ct = 4 * (int)threadIdx.x;
  const int wch0 = warp * 128;
  const int64_t cb = (int64_t)blockIdx.x * 1024 + wch0;
  const int nch = (n - cb < 128) ? (int)((n - cb > 0) ? n - cb : 0) : 128;
  for (int64_t rt = r_begin; rt < r_end; rt += kAtRows) {
    const int64_t rt_end = (rt + kAtRows < r_end) ? rt + kAtRows : r_end;
    if (active) {
      for (int64_t r = rt; r < rt_end; r += 8) {
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = (r + i < rt_end) ? *reinterpret_cast<const float4*>(Z + (r + i) * n + c0) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          __align__(16) __nv_bfloat16 col[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float z = q == 0 ? v[i].x : q == 1 ? v[i].y : q == 2 ? v[i].z : v[i].w;
            col[i] = __float2bfloat16_rn(fmaxf(z, 0.f));
          }
          // (kAtPitch = 36 elements: a row of the tile starts 8-byte aligned, so two 8-byte stores)
          uint2* dst = reinterpret_cast<uint2*>(&zt_tile[(ct + q) * kAtPitch + (int)(r - rt)]);
          dst[0] = *reinterpret_cast<const uint2*>(col);
          dst[1] = *reinterpret_cast<const uint2*>(col + 4);
        }
      }
    }
    __syncwarp();
    const int rows_here = (int)(rt_end - rt);
    for (int e = lane; e < nch * (kAtRows / 8); e += 32) {
      const int ch = e / (kAtRows / 8), piece = e % (kAtRows / 8);
      const int row = row_of[warp][ch];
      if (row < 0) continue;
      const __nv_bfloat16* src = &zt_tile[(wch0 + ch) * kAtPitch + piece * 8];
      __nv_bfloat16* dst = Ht + (int64_t)row * ldt + rt + piece * 8;
      if (piece * 8 + 8 <= rows_here) {
        const uint2 lo = *reinterpret_cast<const uint2*>(src), hi = *reinterpret_cast<const uint2*>(src + 4);
        *reinterpret_cast<uint4*>(dst) = make_uint4(lo.x, lo.y, hi.x, hi.y);
      } else {
        for (int q = 0; q < 8; ++q)
          if (piece * 8 + q < rows_here) dst[q] = src[q];
      }
    }
    __syncwarp();
  }
}

// init pass: A = phi(Z) in storage dtype, optional storage copy of Z, |A| column partials.
// A thread owns 4 consecutive channels and walks its rows four at a time (16-byte loads of all four rows in flight
// before the first store, as in the fused update); |A| is summed in fp32 over the four rows of a round and in fp64
// across rounds.
__global__ void __launch_bounds__(256) init_act_kernel(const float* __restrict__ Z, float* gate_io, void* A_out,
                                                       void* Zb_out, int32_t out_dtype, int64_t T, int64_t n,
                                                       double* absA_part, int32_t row_blocks) {
  const int64_t c0 = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (c0 >= n) return;
  const int64_t rows_per = ceil_div(T, (int64_t)row_blocks);
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per;
  const int64_t r_end = (r_begin + rows_per < T) ? r_begin + rows_per : T;
  const int cnt = (n - c0 >= 4) ? 4 : (int)(n - c0);
  const bool vec = (n % 4 == 0);
  double cs[4] = {0.0, 0.0, 0.0, 0.0};
  auto load4 = [&](const float* base, int64_t e, float* v) {
    if (vec) {
      const float4 x = *reinterpret_cast<const float4*>(base + e);
      v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) v[q] = (q < cnt) ? base[e + q] : 0.f;
    }
  };
  auto store_out = [&](void* base, int64_t e, const float* v) {
    if (vec) {
      store4(base, out_dtype, e, v);
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (q < cnt) {
          if (out_dtype == SP_BF16) reinterpret_cast<__nv_bfloat16*>(base)[e + q] = __float2bfloat16_rn(v[q]);
          else reinterpret_cast<float*>(base)[e + q] = v[q];
        }
      }
    }
  };
  for (int64_t r0 = r_begin; r0 < r_end; r0 += 4) {
    float z[4][4], zg[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t r = r0 + i;
      if (r < r_end) {
        load4(Z, r * n + c0, z[i]);
        if (gate_io) load4(gate_io, r * n + c0, zg[i]);
      }
    }
    float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t r = r0 + i;
      if (r >= r_end) continue;
      const int64_t e = r * n + c0;
      float a[4];
      if (gate_io) {       // gated module: the buffer holds the gate pre-activation, SiLU of it replaces it
        float gt[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          gt[q] = zg[i][q] / (1.f + expf(-zg[i][q]));
          a[q] = gt[q] * z[i][q];
        }
        if (vec) {
          *reinterpret_cast<float4*>(gate_io + e) = make_float4(gt[0], gt[1], gt[2], gt[3]);
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (q < cnt) gate_io[e + q] = gt[q];
        }
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) a[q] = fmaxf(z[i][q], 0.f);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) ps[q] += (q < cnt) ? fabsf(a[q]) : 0.f;
      store_out(A_out, e, a);
      if (Zb_out) store_out(Zb_out, e, z[i]);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) cs[q] += (double)ps[q];
  }
  if (absA_part)
    for (int q = 0; q < cnt; ++q) absA_part[(int64_t)blockIdx.y * n + c0 + q] = cs[q];
}

// out[j] (+)= sum_r part[r, j]: a block takes 32 columns, its 8 warps take every 8th row block (four loads in flight
// each), then the 8 partial sums of a column are added in a fixed order.
__global__ void __launch_bounds__(256) reduce_col_partials_kernel(const double* __restrict__ part, int32_t row_blocks,
                                                                  int64_t n, double* out, int acc) {
  __shared__ double sm[8][33];
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int64_t j = (int64_t)blockIdx.x * 32 + cx;
  double s = 0.0;
  if (j < n) {
    int r = ry;
    for (; r + 24 < row_blocks; r += 32) {
      const double v0 = part[(int64_t)r * n + j], v1 = part[(int64_t)(r + 8) * n + j];
      const double v2 = part[(int64_t)(r + 16) * n + j], v3 = part[(int64_t)(r + 24) * n + j];
      s += v0; s += v1; s += v2; s += v3;
    }
    for (; r < row_blocks; r += 8) s += part[(int64_t)r * n + j];
  }
  sm[ry][cx] = s;
  __syncthreads();
  if (ry == 0 && j < n) {
    double tot = acc ? out[j] : 0.0;
#pragma unroll
    for (int q = 0; q < 8; ++q) tot += sm[q][cx];
    out[j] = tot;
  }
}

__global__ void reduce_report_kernel(const double* partial, int nblocks, sp_step_report* rep, int acc, double alpha) {
  __shared__ double sm[32];
  double s[4] = {0.0, 0.0, 0.0, 0.0};
  for (int i = threadIdx.x; i < nblocks; i += blockDim.x)
    for (int f = 0; f < 4; ++f) s[f] += partial[(int64_t)i * 4 + f];
  for (int f = 0; f < 4; ++f) {
    const double r = block_sum<double>(s[f], sm);
    if (threadIdx.x == 0) {
      double* dst = f == 0 ? &rep->res_act : (f == 1 ? &rep->z_sq : (f == 2 ? &rep->a_sq : &rep->res_in));
      *dst = (acc ? *dst : 0.0) + (f == 3 ? alpha * r : r);
    }
  }
}

// out[0] (+)= scale * sum x^2 over a [rows, cols] fp32 matrix: block partials, then one block adds them in order
__global__ void __launch_bounds__(256) sumsq_partial_kernel(const float* __restrict__ x, int64_t ld, int64_t rows,
                                                            int64_t cols, double* part) {
  __shared__ double sm[32];
  double s = 0.0;
  const int64_t total = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const float v = x[(e / cols) * ld + (e % cols)];
    s += (double)v * (double)v;
  }
  const double r = block_sum<double>(s, sm);
  if (threadIdx.x == 0) part[blockIdx.x] = r;
}
__global__ void sumsq_finish_kernel(const double* part, int nblocks, double scale, double* out, int acc) {
  __shared__ double sm[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < nblocks; i += blockDim.x) s += part[i];
  const double r = block_sum<double>(s, sm);
  if (threadIdx.x == 0) out[0] = (acc ? out[0] : 0.0) + scale * r;
}

__global__ void init_report_kernel(sp_step_report* rep, const double* rho1, const double* rho2, double kept,
                                   const int32_t* reused, const int32_t* scaled) {
  rep->res_act = 0.0;
  rep->res_out = nan("");
  rep->res_in = 0.0;
  rep->z_sq = 0.0;
  rep->a_sq = 0.0;
  rep->rho1_eff = rho1 ? rho1[0] : 0.0;
  rep->rho2_eff = rho2 ? rho2[0] : 0.0;
  rep->kept = kept;
  rep->factor_reused = (reused != nullptr && reused[0] != 0) ? 1.0 : 0.0;
  rep->pruned_scaled = (scaled != nullptr && scaled[0] != 0) ? 1.0 : 0.0;
}

// per-column sum |x| and sum x^2 of a [T, C] chunk: grid (col blocks of 256, row blocks) -> scratch, then reduced
__global__ void column_stats_kernel(const void* X, int32_t dt, int64_t ld, int64_t T, int64_t C, double* scratch,
                                    int32_t row_blocks) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const int64_t rows_per = ceil_div(T, (int64_t)row_blocks);
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per;
  const int64_t r_end = (r_begin + rows_per < T) ? r_begin + rows_per : T;
  double s1 = 0.0, s2 = 0.0;
  for (int64_t r = r_begin; r < r_end; ++r) {
    const double v = (double)ld_any(X, dt, r * ld + c);
    s1 += fabs(v);
    s2 += v * v;
  }
  scratch[((int64_t)blockIdx.y * C + c) * 2 + 0] = s1;
  scratch[((int64_t)blockIdx.y * C + c) * 2 + 1] = s2;
}

__global__ void column_stats_reduce_kernel(const double* scratch, int32_t row_blocks, int64_t C, double* rowstats) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  double s1 = rowstats[c * 2 + 0], s2 = rowstats[c * 2 + 1];
  for (int r = 0; r < row_blocks; ++r) {
    s1 += scratch[((int64_t)r * C + c) * 2 + 0];
    s2 += scratch[((int64_t)r * C + c) * 2 + 1];
  }
  rowstats[c * 2 + 0] = s1;
  rowstats[c * 2 + 1] = s2;
}

inline int grid_for(int64_t total, int threads, int per_thread = 1) {
  int64_t b = ceil_div(total, (int64_t)threads * per_thread);
  const int64_t cap = 148 * 16;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (int)b;
}

}  // namespace

cudaError_t convert_matrix(const void* src, int32_t sdt, int64_t lds, void* dst, int32_t ddt, int64_t ldd,
                           int64_t rows, int64_t cols, cudaStream_t stream) {
  if (rows * cols == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  convert_kernel<<<grid_for(rows * cols, 256), 256, 0, stream>>>(src, sdt, lds, dst, ddt, ldd, rows, cols);
  return cudaGetLastError();
}

template <typename TD>
cudaError_t transpose_convert(const float* src, int64_t lds, int64_t rows, int64_t cols, TD* dst, int64_t ldd,
                              cudaStream_t stream) {
  if (rows * cols == 0) return cudaSuccess;
  dim3 grid((unsigned)ceil_div(cols, 32), (unsigned)ceil_div(rows, 32));
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  transpose_convert_kernel<TD><<<grid, dim3(32, 8), 0, stream>>>(src, lds, rows, cols, dst, ldd);
  return cudaGetLastError();
}
template cudaError_t transpose_convert<float>(const float*, int64_t, int64_t, int64_t, float*, int64_t, cudaStream_t);
template cudaError_t transpose_convert<double>(const float*, int64_t, int64_t, int64_t, double*, int64_t,
                                               cudaStream_t);
template cudaError_t transpose_convert<__nv_bfloat16>(const float*, int64_t, int64_t, int64_t, __nv_bfloat16*,
                                                      int64_t, cudaStream_t);

cudaError_t split3_bf16(const float* src, int64_t lds, int64_t rows, int64_t cols, int64_t kpad, void* dst,
                        cudaStream_t stream) {
  if (rows * kpad == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)rows * cols * 10.0, stream);
  count_launch();
  split3_bf16_kernel<<<grid_for(rows * kpad, 256), 256, 0, stream>>>(src, lds, rows, cols, kpad,
                                                                     reinterpret_cast<__nv_bfloat16*>(dst));
  return cudaGetLastError();
}

cudaError_t split_bf16(const float* src, int64_t lds, const int32_t* row_idx, int64_t rows, int64_t cols, int64_t kpad,
                       void* dst, cudaStream_t stream) {
  if (rows * kpad == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  split_bf16_kernel<<<grid_for(rows * kpad, 256), 256, 0, stream>>>(src, lds, row_idx, rows, cols, kpad,
                                                                     reinterpret_cast<__nv_bfloat16*>(dst));
  return cudaGetLastError();
}

cudaError_t symmetrize_lower(float* G, int64_t n, int64_t ld, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  const unsigned nb = (unsigned)ceil_div(n, 32);
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  symmetrize_kernel<<<dim3(nb, nb), dim3(32, 8), 0, stream>>>(G, n, ld);
  return cudaGetLastError();
}

template <typename T>
cudaError_t load_spd(const float* G, int64_t ldg, int64_t n, const double* rho_dev, T* dst, int64_t ldd,
                     cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  load_spd_kernel<T><<<grid_for(n * n, 256), 256, 0, stream>>>(G, ldg, nullptr, n, rho_dev, dst, ldd, skip_flag());
  return cudaGetLastError();
}
template <typename T>
cudaError_t load_spd_gather(const float* G, int64_t ldg, const int32_t* idx, int64_t k, const double* rho_dev, T* dst,
                            int64_t ldd, cudaStream_t stream) {
  if (k == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  load_spd_kernel<T><<<grid_for(k * k, 256), 256, 0, stream>>>(G, ldg, idx, k, rho_dev, dst, ldd, skip_flag());
  return cudaGetLastError();
}
template <typename T>
cudaError_t gather_cols(const float* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k, T* dst,
                        int64_t ldd, cudaStream_t stream) {
  if (rows * k == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  gather_cols_kernel<T><<<grid_for(rows * k, 256), 256, 0, stream>>>(src, lds, idx, rows, k, dst, ldd, skip_flag());
  return cudaGetLastError();
}
cudaError_t copy_cols_padded(const float* src, int64_t lds, int64_t rows, int64_t k, int64_t kpad, float* dst,
                             cudaStream_t stream) {
  if (rows * kpad == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  copy_cols_padded_kernel<<<grid_for(rows * kpad, 256), 256, 0, stream>>>(src, lds, rows, k, kpad, dst);
  return cudaGetLastError();
}
cudaError_t gather_rows(const float* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t cols, float* dst,
                        int64_t ldd, cudaStream_t stream) {
  if (rows * cols == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  gather_rows_kernel<<<grid_for(rows * cols, 256), 256, 0, stream>>>(src, lds, idx, rows, cols, dst, ldd);
  return cudaGetLastError();
}

template <typename T>
cudaError_t scatter_cols(const T* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k, int64_t n,
                         float* dst, int64_t ldd, cudaStream_t stream) {
  if (rows * n == 0) return cudaSuccess;
  if (idx) {
    ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
    count_launch();
    fill_zero_kernel<<<grid_for(rows * n, 256), 256, 0, stream>>>(dst, ldd, rows, n, skip_flag());
  }
  if (rows * k == 0) return cudaGetLastError();
  count_launch();
  scatter_cols_kernel<T><<<grid_for(rows * k, 256), 256, 0, stream>>>(src, lds, idx, rows, k, dst, ldd,
                                                                      skip_flag());
  return cudaGetLastError();
}
#define SP_INST(T)                                                                                                  \
  template cudaError_t load_spd<T>(const float*, int64_t, int64_t, const double*, T*, int64_t, cudaStream_t);      \
  template cudaError_t load_spd_gather<T>(const float*, int64_t, const int32_t*, int64_t, const double*, T*,       \
                                          int64_t, cudaStream_t);                                                   \
  template cudaError_t gather_cols<T>(const float*, int64_t, const int32_t*, int64_t, int64_t, T*, int64_t,        \
                                      cudaStream_t);                                                                \
  template cudaError_t scatter_cols<T>(const T*, int64_t, const int32_t*, int64_t, int64_t, int64_t, float*,       \
                                       int64_t, cudaStream_t);
SP_INST(float)
SP_INST(double)
#undef SP_INST

cudaError_t effective_ridge(const float* G, int64_t ldg, int64_t n, double rho, int rel, double* rho_out,
                            cudaStream_t stream) {
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  effective_ridge_kernel<<<1, 1024, 0, stream>>>(G, ldg, n, rho, rel, rho_out);
  return cudaGetLastError();
}

cudaError_t build_group_map(const uint8_t* mask, int64_t n, int32_t* grp_base, uint8_t* grp_mask, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  group_map_kernel<<<1, 1024, 0, stream>>>(mask, n, grp_base, grp_mask);
  return cudaGetLastError();
}

cudaError_t launch_prep_h(const float* Z, const float* U, const float* gate, void* H, int32_t hdt, int64_t T,
                          int64_t n, int64_t ldh, int64_t k, const int32_t* idx, cudaStream_t stream, int64_t lo_off) {
  if (T * ldh == 0) return cudaSuccess;
  if (lo_off > 0 && (hdt != SP_BF16 || lo_off % 8 != 0 || 2 * lo_off > ldh)) return cudaErrorInvalidValue;
  const int64_t ncols = lo_off > 0 ? lo_off : ldh;
  // algorithmic bytes: Z (and U) read once, the kept part written once (twice when it is split); a conditional
  // launch (SkipScope) is not counted: whether it moves anything is decided on the device
  ProfScope prof(PK_PREP_H, 0.0,
                 skip_flag() != nullptr ? 0.0 :
                 (double)T * ((double)n * (U ? 8.0 : 4.0) +
                              (double)k * ((hdt == SP_BF16 ? (lo_off > 0 ? 4.0 : 2.0) : 4.0) + (gate ? 4.0 : 0.0))),
                 stream);
  const unsigned gx = (unsigned)ceil_div(ncols, (int64_t)(8 * 256));
  int64_t rb = ceil_div((int64_t)148 * 16, (int64_t)gx);
  if (rb > T) rb = T;
  if (rb > 65535) rb = 65535;
  const int32_t rows_per = (int32_t)ceil_div(T, rb);
  count_launch();
  prep_h_kernel<<<dim3(gx, (unsigned)ceil_div(T, (int64_t)rows_per)), 256, 0, stream>>>(Z, U, gate, H, hdt, T, n, ldh, ncols, lo_off,
                                                                                        k, idx, rows_per, skip_flag());
  return cudaGetLastError();
}

int fused_update_grid(int64_t T, int64_t n, int* row_blocks) {
  const int col_blocks = (int)ceil_div(n, 1024);
  int rb = (148 * 16 + col_blocks - 1) / col_blocks;
  if (rb > T) rb = (int)T;
  if (rb < 1) rb = 1;
  if (rb > 65535) rb = 65535;
  *row_blocks = rb;
  return col_blocks * rb;
}

// Grid of the form that also writes the next step's operands: column blocks of kNextChannels channels, row blocks of
// a multiple of kNextTiles * kAtRows rows.  The rows per block are chosen so that the blocks fill whole waves of the
// 2 x 148 resident blocks as nearly as possible (at n = 28672 the plain rule "16 blocks per SM" left the last of 8.3
// waves 30 % full); the number of row blocks never exceeds fused_update_next_row_cap(n), which sizes the partial sums.
int fused_update_next_partial_rows(int row_blocks) { return kNextTiles * row_blocks; }
int fused_update_next_row_cap(int64_t n) {
  const int64_t col_blocks = ceil_div(n, (int64_t)kNextChannels);
  return (int)std::min<int64_t>(65535, ceil_div((int64_t)148 * 32, col_blocks) + 1);
}
int64_t fused_update_next_max_blocks(int64_t n) {
  return ceil_div(n, (int64_t)kNextChannels) * fused_update_next_row_cap(n);
}
int fused_update_next_grid(int64_t T, int64_t n, int* row_blocks) {
  const int64_t col_blocks = ceil_div(n, (int64_t)kNextChannels);
  const int64_t unit = (int64_t)kNextTiles * kAtRows, slots = 2 * 148, cap = fused_update_next_row_cap(n);
  int64_t best_rb = 1, best_span = -1;
  for (int64_t r = unit * ceil_div(T, unit); r >= unit; r -= unit) {
    const int64_t rb = ceil_div(T, r);
    if (rb > cap) break;
    const int64_t span = ceil_div(col_blocks * rb, slots) * r;     // waves x rows per block
    if (best_span < 0 || span < best_span) { best_span = span; best_rb = rb; }
    if (r > 64 * unit) r -= (r / (64 * unit) - 1) * unit;          // (coarser steps among very tall blocks)
  }
  *row_blocks = (int)best_rb;
  return (int)(col_blocks * best_rb);
}

static cudaError_t launch_fused_update_next(const UpdateArgs& a, cudaStream_t stream) {
  if (a.U || a.gate || a.n % 4 != 0 || a.ldt % 8 != 0 || !a.At_out || !a.Zt_out || !a.Ht_out || !a.at_kept_first ||
      a.out_dtype != SP_BF16)
    return cudaErrorInvalidValue;
  dim3 grid((unsigned)ceil_div(a.n, (int64_t)kNextChannels), (unsigned)a.row_blocks);
  // per row: Z read and written, A^T written; z1 and D read, Z^T and h^T written on the kept channels (the pruned rows
  // of Z^T, written only after a mask change, are not counted)
  ProfScope prof(PK_FUSED_UPDATE, 0.0, (double)a.T * ((double)a.n * 10.0 + (double)a.k * 12.0), stream);
  count_launch();
  const bool pz = a.z_rule == SP_Z_PAPER;
  void (*fn)(UpdateArgs) = pz ? &fused_update_next_kernel<SP_Z_PAPER> : &fused_update_next_kernel<SP_Z_EXACT>;
  cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kNextTileBytes);
  if (e != cudaSuccess) return e;
  fn<<<grid, 256, kNextTileBytes, stream>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_fused_update(const UpdateArgs& a, cudaStream_t stream) {
  if (a.T * a.n == 0) return cudaSuccess;
  if (a.Zt_out || a.Ht_out) return launch_fused_update_next(a, stream);
  dim3 grid((unsigned)ceil_div(a.n, 1024), (unsigned)a.row_blocks);
  // algorithmic bytes per row: Z (and U) read and written, A and the storage copy of Z written, z1 and D read on the
  // kept channels
  const double esz = a.out_dtype == SP_BF16 ? 2.0 : 4.0;
  const double per_n = 8.0 + (a.U ? 8.0 : 0.0) + esz + (a.Zb_out ? esz : 0.0) + (a.gate ? 4.0 : 0.0);
  ProfScope prof(PK_FUSED_UPDATE, 0.0, (double)a.T * ((double)a.n * per_n + (double)a.k * 8.0), stream);
  count_launch();
  const bool pz = a.z_rule == SP_Z_PAPER;
  // the transposed-A tile of one block is above the default 48 KB limit
  const size_t smem = a.At_out ? kAtTileBytes : 0;
  void (*fn)(UpdateArgs) = nullptr;
  if (a.gate) fn = a.U ? &fused_update_kernel<true, kZGated> : &fused_update_kernel<false, kZGated>;
  else if (a.U) fn = pz ? &fused_update_kernel<true, SP_Z_PAPER> : &fused_update_kernel<true, SP_Z_EXACT>;
  else fn = pz ? &fused_update_kernel<false, SP_Z_PAPER> : &fused_update_kernel<false, SP_Z_EXACT>;
  if (smem) {
    cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn),
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  fn<<<grid, 256, smem, stream>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gather_ht(const float* Z, int64_t T, int64_t n, int64_t k, const int32_t* grp_base,
                             const uint8_t* grp_mask, void* Ht, int64_t ldt, cudaStream_t stream) {
  if (T * n == 0) return cudaSuccess;
  if (n % 4 != 0 || ldt % 8 != 0) return cudaErrorInvalidValue;
  int row_blocks = 1;
  fused_update_grid(T, n, &row_blocks);
  dim3 grid((unsigned)ceil_div(n, (int64_t)1024), (unsigned)row_blocks);
  const int32_t* skip = skip_flag();
  ProfScope prof(skip ? PK_CONDITIONAL : PK_PREP_H, 0.0, skip ? 0.0 : (double)T * ((double)n * 4.0 + (double)k * 2.0),
                 stream);
  count_launch();
  cudaError_t e = cudaFuncSetAttribute(gather_ht_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kAtTileBytes);
  if (e != cudaSuccess) return e;
  gather_ht_kernel<<<grid, 256, kAtTileBytes, stream>>>(Z, T, n, k, grp_base, grp_mask,
                                                       reinterpret_cast<__nv_bfloat16*>(Ht), ldt, row_blocks, skip);
  return cudaGetLastError();
}

cudaError_t launch_init_act(const float* Z, float* gate_io, void* A_out, void* Zb_out, int32_t out_dtype, int64_t T,
                            int64_t n, double* absA_part, int32_t row_blocks, cudaStream_t stream) {
  if (T * n == 0) return cudaSuccess;
  dim3 grid((unsigned)ceil_div(n, 1024), (unsigned)row_blocks);
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  init_act_kernel<<<grid, 256, 0, stream>>>(Z, gate_io, A_out, Zb_out, out_dtype, T, n, absA_part, row_blocks);
  return cudaGetLastError();
}

cudaError_t reduce_col_partials(const double* part, int32_t row_blocks, int64_t n, double* out, bool accumulate,
                                cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  reduce_col_partials_kernel<<<(unsigned)ceil_div(n, (int64_t)32), 256, 0, stream>>>(part, row_blocks, n, out,
                                                                                    accumulate ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t reduce_report(const double* partial, int nblocks, sp_step_report* rep, bool accumulate, double alpha,
                          cudaStream_t stream) {
  count_launch();
  reduce_report_kernel<<<1, 256, 0, stream>>>(partial, nblocks, rep, accumulate ? 1 : 0, alpha);
  return cudaGetLastError();
}

cudaError_t sumsq_accumulate(const float* x, int64_t ld, int64_t rows, int64_t cols, double scale, double* out,
                             bool accumulate, double* scratch, cudaStream_t stream) {
  if (rows * cols == 0) return cudaSuccess;
  ProfScope prof(PK_ELEMENTWISE, 0.0, (double)rows * cols * 4.0, stream);
  const int nb = kSumsqBlocks;
  count_launch(2);
  sumsq_partial_kernel<<<nb, 256, 0, stream>>>(x, ld, rows, cols, scratch);
  sumsq_finish_kernel<<<1, 256, 0, stream>>>(scratch, nb, scale, out, accumulate ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t init_report(sp_step_report* rep, const double* rho1, const double* rho2, double kept,
                        const int32_t* reused, const int32_t* scaled, cudaStream_t stream) {
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  init_report_kernel<<<1, 1, 0, stream>>>(rep, rho1, rho2, kept, reused, scaled);
  return cudaGetLastError();
}

cudaError_t column_stats(const void* X, int32_t dt, int64_t ld, int64_t T, int64_t C, double* rowstats,
                         double* scratch, cudaStream_t stream) {
  if (T * C == 0) return cudaSuccess;
  const int rb = column_stats_row_blocks(T, C);
  dim3 grid((unsigned)ceil_div(C, 256), (unsigned)rb);
  ProfScope prof(PK_ELEMENTWISE, 0.0, 0.0, stream);
  count_launch();
  column_stats_kernel<<<grid, 256, 0, stream>>>(X, dt, ld, T, C, scratch, rb);
  count_launch();
  column_stats_reduce_kernel<<<(unsigned)ceil_div(C, 256), 256, 0, stream>>>(scratch, rb, C, rowstats);
  return cudaGetLastError();
}

int column_stats_row_blocks(int64_t T, int64_t C) {
  const int64_t cb = ceil_div(C, 256);
  int64_t rb = ceil_div(148 * 4, cb);
  if (rb > T) rb = T;
  if (rb < 1) rb = 1;
  return (int)rb;
}

}  // namespace sp
