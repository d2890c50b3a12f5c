// C-ABI entry points of libsp and the host-side orchestration of the per-module ADMM step.
#include <math.h>
#include <string.h>

#include <mutex>

#include "sp_common.cuh"

using namespace sp;

#define CU(x)                                  \
  do {                                         \
    if ((x) != cudaSuccess) return SP_ERR_CUDA; \
  } while (0)
#define SPCHK(x)               \
  do {                         \
    sp_status _s = (x);        \
    if (_s != SP_OK) return _s; \
  } while (0)

namespace {

constexpr int64_t kDefaultChunk = 32768;
// SM pairs given to the z1 products that run beside the kept-support recovery (of 74 on a B200): 40 to 66 pairs
// measured the same within noise.
constexpr int kZ1AheadPairs = 58;

struct MatRef {
  const void* ptr;
  int32_t dtype;
  int64_t ld;
};

// C[M,N] = alpha * sum_k A(i,k) B(k,j) + beta * Cin.
//   a_kmajor: A stored [M,K] (ld) else [K,M];  b_kmajor: B stored [N,K] (ld) else [K,N].
// bf16 operands go to the tensor-core kernel when its alignment rules hold; everything else (and the fp32 mode,
// which accumulates in fp64) runs on the CUDA-core kernel.
sp_status contract(int64_t M, int64_t N, int64_t K, double alpha, MatRef A, bool a_kmajor, MatRef B, bool b_kmajor,
                   double beta, MatRef Cin, MatRef C, bool lower_only, bool acc64, bool allow_tc, int32_t* status,
                   cudaStream_t stream) {
  if (M <= 0 || N <= 0) return SP_OK;
  Operand cin{Cin.ptr, Cin.dtype, Cin.ld, 1};
  OutOperand out{const_cast<void*>(C.ptr), C.dtype, C.ld};
  if (allow_tc && A.dtype == SP_BF16 && B.dtype == SP_BF16 && K > 0 && C.dtype != SP_F64 &&
      (beta == 0.0 || Cin.dtype != SP_F64)) {
    TcOperand ta{A.ptr, A.ld, a_kmajor}, tb{B.ptr, B.ld, b_kmajor};
    if (gemm_tc_supported(M, N, K, ta, tb)) return gemm_tc(M, N, K, (float)alpha, ta, tb, (float)beta, cin, out,
                                                           lower_only, status, stream);
  }
  Operand a{A.ptr, A.dtype, a_kmajor ? A.ld : 1, a_kmajor ? 1 : A.ld};
  Operand b{B.ptr, B.dtype, b_kmajor ? 1 : B.ld, b_kmajor ? B.ld : 1};
  CU(gemm_simt(M, N, K, alpha, a, b, beta, cin, out, lower_only, acc64, stream));
  return SP_OK;
}

// C[M,N] = A W^T with fp32 weights W[N,K]: on the tensor cores W is split into bf16 hi + lo parts stored side by side
// ([N, 2*kpad]) so that no weight bit beyond ~16 is lost; A (bf16, [M,K], ld) is read once per part.
// Falls back to the CUDA-core kernel (fp32 W as is) when the tensor-core path's alignment rules do not hold.
int64_t split_kpad(int64_t K) { return (K + 63) / 64 * 64; }

sp_status contract_split_weights(int64_t M, int64_t N, int64_t K, MatRef A, const void* Wsplit, MatRef Wf32, MatRef C,
                                 int32_t* status, cudaStream_t stream, int max_pairs = 0) {
  if (M <= 0 || N <= 0) return SP_OK;
  const int64_t kp = split_kpad(K);
  TcOperand ta{A.ptr, A.ld, true}, tb{Wsplit, 2 * kp, true};
  tb.kext = 2 * kp;
  OutOperand out{const_cast<void*>(C.ptr), C.dtype, C.ld};
  Operand cin{C.ptr, C.dtype, C.ld, 1};
  if (Wsplit && A.dtype == SP_BF16 && gemm_tc_supported(M, N, K, ta, tb)) {
    TcSegments sg;
    sg.nseg = 2;            // hi part, then lo part, against the same A tile
    sg.b_k[1] = (int32_t)kp;
    return gemm_tc(M, N, K, 1.f, ta, tb, 0.f, cin, out, false, status, stream, &sg, 2.0 * (double)M * N * K,
                   max_pairs);
  }
  if (Wf32.ptr) return contract(M, N, K, 1.0, A, true, Wf32, true, 0.0, C, C, false, false, false, status, stream);
  // no fp32 copy at hand: hi and lo parts one after the other on the CUDA cores
  MatRef hi{Wsplit, SP_BF16, 2 * kp}, lo{reinterpret_cast<const __nv_bfloat16*>(Wsplit) + kp, SP_BF16, 2 * kp};
  SPCHK(contract(M, N, K, 1.0, A, true, hi, true, 0.0, C, C, false, false, false, status, stream));
  return contract(M, N, K, 1.0, A, true, lo, true, 1.0, C, C, false, false, false, status, stream);
}

struct Carver {
  uint8_t* base;
  size_t off = 0;
  explicit Carver(void* p) : base(reinterpret_cast<uint8_t*>(p)) {}
  template <typename T>
  T* take(size_t count) {
    off = align_up(off, 256);
    T* p = reinterpret_cast<T*>(base + off);
    off += count * sizeof(T);
    return p;
  }
  void* take_bytes(size_t bytes) {
    off = align_up(off, 256);
    void* p = base + off;
    off += bytes;
    return p;
  }
};

size_t dinv_elems(int64_t n) {
  const size_t simt = (size_t)ceil_div(n, (int64_t)kCholNB) * kCholNB * kCholNB;
  const size_t tc = ((size_t)ceil_div(n, (int64_t)kCholTcNB) + 1) * 2 * kCholTcNB * kCholTcNB;   // + scratch pair
  return simt > tc ? simt : tc;
}

// Buffers of the regularised solve for systems up to nmax with up to mmax right-hand sides.
struct SolveBufs {
  void* Gs;
  void* dinv;
  int32_t* idx;
  double* rho;  // [4] device scalars
  void* P;      // fp32 path: bf16 parts of the Cholesky factor
  void* Xs;     // fp32 path: bf16 parts of one block column of right-hand sides
};

SolveBufs carve_solve(Carver& c, int64_t nmax, int64_t mmax, size_t tsize) {
  SolveBufs b;
  b.rho = c.take<double>(4);
  b.idx = c.take<int32_t>((size_t)nmax);
  // the system matrix and, right behind its nn x nn elements, the right-hand sides (one [nn + m, nn] array)
  b.Gs = c.take_bytes((size_t)(nmax + mmax) * nmax * tsize);
  b.dinv = c.take_bytes(dinv_elems(nmax) * tsize);
  b.P = nullptr;
  b.Xs = nullptr;
  if (tsize == 4) {
    const size_t np = (size_t)chol_tc_pad(nmax);
    b.P = c.take_bytes((np + (size_t)mmax) * 3 * np * 2);
    const size_t rows = (size_t)(nmax > mmax ? nmax : mmax);   // either dimension may be the right-hand-side count
    b.Xs = c.take_bytes(2 * rows * 3 * kCholTcNB * 2);
  }
  return b;
}

// Copy of the forward-substituted right-hand sides on the leading k columns of a system (tensor-core path): with it
// and the factor's leading block the system restricted to its first k unknowns is solved by a backward sweep alone.
struct LeadSave {
  float* Y;       // [m, kpad] dense, columns k..kpad zero
  int64_t k, kpad;
};

// W[m, n_full] = R[:, idx] (G[idx, idx] + rho I)^-1 scattered back to the idx columns (idx == nullptr: identity).
// conditional: the call runs under a SkipScope (its work is not counted in the profile's flops).
template <typename T>
sp_status ridge_core(const float* R, int64_t ldr, const float* G, int64_t ldg, int64_t m, int64_t n_full,
                     const int32_t* idx, int64_t k, const double* rho_dev, float* W, int64_t ldw, SolveBufs& b,
                     int32_t* status, cudaStream_t stream, const SolveAssist* assist = nullptr,
                     bool split_lookahead = false, const LeadSave* save = nullptr, bool conditional = false) {
  const int64_t nn = idx ? k : n_full;
  ProfScope prof(PK_SOLVE, conditional ? 0.0 : (double)nn * nn * nn / 3.0 + 2.0 * (double)m * nn * nn, 0.0, stream);
  T* Gs = reinterpret_cast<T*>(b.Gs);
  T* dinv = reinterpret_cast<T*>(b.dinv);
  T* Rs = Gs + (size_t)nn * nn;     // the right-hand sides sit right below the system matrix, same leading dimension
  if (idx) CU(load_spd_gather<T>(G, ldg, idx, nn, rho_dev, Gs, nn, stream));
  else CU(load_spd<T>(G, ldg, nn, rho_dev, Gs, nn, stream));
  if constexpr (sizeof(T) == 4) {
    // the right-hand sides ride through the factorisation as m more rows (their forward substitution); the solve
    // proper is then only the backward sweep
    CU(gather_cols<T>(R, ldr, idx, m, nn, Rs, nn, stream));
    SPCHK(potrf_lower_tc(Gs, nn, nn, dinv, b.P, status, stream, assist, m, split_lookahead));
    if (save) CU(copy_cols_padded(Rs, nn, m, save->k, save->kpad, save->Y, stream));
    SPCHK(potrs_right_tc(Rs, m, nn, nn, b.P, dinv, b.Xs, status, stream, assist, true, Gs, nn));
  } else {
    CU(potrf_lower<T>(Gs, nn, nn, dinv, status, stream));
    CU(gather_cols<T>(R, ldr, idx, m, nn, Rs, nn, stream));
    CU(potrs_right<T>(Rs, m, nn, nn, Gs, nn, dinv, stream));
  }
  CU(scatter_cols<T>(Rs, nn, idx, m, nn, n_full, W, ldw, stream));
  return SP_OK;
}

__global__ void expand_group_index_kernel(const int32_t* unit_idx, int64_t k_units, int group, int32_t* col_idx) {
  const int64_t total = k_units * group;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x)
    col_idx[e] = unit_idx[e / group] * group + (int32_t)(e % group);
}

// A library-owned side stream per device: independent parts of one call (the W1 recovery next to the W2 recovery)
// are forked onto it from the caller's stream and joined back with events, so the call stays asynchronous and
// ordered on the caller's stream.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, z1_done = nullptr;
  SolveAssist assist_main{}, assist_side{};   // helpers of the solves on the caller's stream / on `stream`
};
bool make_assist(SolveAssist& a) {
  return cudaStreamCreateWithFlags(&a.stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.panel_done, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.rest_done[0], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.rest_done[1], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.near_done, cudaEventDisableTiming) == cudaSuccess &&
         cudaStreamCreateWithFlags(&a.far_stream, cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.far_go, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.far_done[0], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&a.far_done[1], cudaEventDisableTiming) == cudaSuccess;
}
SideStream* side_stream() {
  static SideStream table[64];
  static bool failed[64] = {};
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> guard(mu);
  if (failed[dev]) return nullptr;
  SideStream& ss = table[dev];
  if (!ss.stream) {
    if (cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ss.join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ss.z1_done, cudaEventDisableTiming) != cudaSuccess ||
        !make_assist(ss.assist_main) || !make_assist(ss.assist_side)) {
      failed[dev] = true;
      ss.stream = nullptr;
      return nullptr;
    }
  }
  return &ss;
}

// Makes the caller's stream wait for everything queued on the library's
// streams when a call returns early (an error between a fork and its join), so that no library work is ever left
// unordered against the caller's stream.
struct JoinOnExit {
  SideStream* side;
  cudaStream_t s;
  bool armed = true;
  ~JoinOnExit() {
    if (!armed || !side) return;
    cudaStream_t all[5] = {side->stream, side->assist_main.stream, side->assist_side.stream,
                           side->assist_main.far_stream, side->assist_side.far_stream};
    for (cudaStream_t q : all) {
      if (cudaEventRecord(side->join, q) == cudaSuccess) cudaStreamWaitEvent(s, side->join, 0);
    }
  }
};

bool valid_act_dtype(int32_t dt) { return dt == SP_F32 || dt == SP_BF16; }
// the sub-buffers of a workspace are carved at 256-byte offsets and accessed with 16-byte vector and bulk copies
bool misaligned(const void* p, size_t a) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) % a) != 0; }

// ------------------------------------------------------------------------------------------------ workspace plans
struct AdmmPlan {
  int64_t d, n, N, chunk;
  int32_t cdt;
  bool bf16;
  size_t tsize;
  // device buffers
  SolveBufs sb;
  SolveBufs sbA;               // buffers of the W1 recovery (system d, n right-hand sides), which runs concurrently
  float *W1t, *W2t, *Qt, *T0, *Cf;
  float *W2cf, *W1c;           // compact fp32 copies on the kept support: W2[:, S] ([d, kp]) and W1[S, :] ([k, d])
  int32_t* perm;               // channels ordered "kept by the previous mask first" (reuse of the G_A factor)
  int32_t* reuse_flags;        // [0] support changed, [1] support unchanged, [2] kept count of the previous mask;
                               // [4] / [5] channel order changed / unchanged against the last token pass (decay_tag)
  int32_t* grp_base;           // kept-channel map of the elementwise kernels
  uint8_t* grp_mask;
  void *W1b, *W2b, *Qtb;       // bf16 operands on the kept support (bf16 mode only)
  void* W2sb;                  // bf16 hi | lo split of W2[:, S] ([d, 2 * pad64(k)], gated modules)
  void *R1p, *Gip;             // three-part bf16 forms of R1 [n, 3 pad64(d)] and of the cached (G_X + rho1 I)^-1
  void *H, *E, *Ac, *Zb;
  float *D, *z1, *Eo;          // Eo: Ypre - A W2^T of a chunk (objective reporting)
  void* W2fb;                  // bf16 copy of the full W2 (objective reporting)
  float* z1_all;               // [N, kp] behind the planned bytes when the caller's workspace has room for it
  double *partial, *absA_part, *score_scratch;
  int row_blocks, nblocks;
  size_t bytes;
};

AdmmPlan plan_admm(void* ws, int64_t d, int64_t n, int64_t N, int64_t chunk, int32_t cdt) {
  AdmmPlan p;
  p.d = d; p.n = n; p.N = N;
  p.chunk = chunk > 0 ? chunk : kDefaultChunk;
  if (p.chunk > N) p.chunk = N;
  if (p.chunk < 1) p.chunk = 1;
  p.cdt = cdt;
  p.bf16 = cdt == SP_BF16;
  p.tsize = p.bf16 ? 4 : 8;
  const size_t csz = p.bf16 ? 2 : 4;
  Carver c(ws);
  const int64_t nmax = n > d ? n : d;
  p.sb = carve_solve(c, nmax, nmax == n ? d : n, p.tsize);
  p.sbA = carve_solve(c, d, n, p.tsize);
  p.W1t = c.take<float>((size_t)n * d);
  p.W2t = c.take<float>((size_t)n * d);
  p.Qt = c.take<float>((size_t)n * d);
  p.T0 = c.take<float>((size_t)n * d);
  p.Cf = c.take<float>((size_t)d * d);
  p.W2cf = c.take<float>((size_t)n * d + 8 * (size_t)d);
  p.W1c = p.bf16 ? nullptr : c.take<float>((size_t)n * d);
  p.perm = c.take<int32_t>((size_t)n);
  p.reuse_flags = c.take<int32_t>(8);
  p.grp_base = c.take<int32_t>((size_t)ceil_div(n, (int64_t)8));
  p.grp_mask = c.take<uint8_t>((size_t)ceil_div(n, (int64_t)8));
  p.W1b = p.bf16 ? c.take_bytes((size_t)n * 2 * split_kpad(d) * csz) : nullptr;   // hi | lo split of W1
  p.W2b = p.bf16 ? c.take_bytes(((size_t)n + 8) * d * csz) : nullptr;
  p.Qtb = p.bf16 ? c.take_bytes((size_t)n * 2 * split_kpad(d) * csz) : nullptr;   // room for the hi | lo form
  p.W2sb = p.bf16 ? c.take_bytes((size_t)d * 2 * split_kpad(n) * csz) : nullptr;
  p.R1p = p.bf16 ? c.take_bytes((size_t)n * 3 * split_kpad(d) * csz) : nullptr;
  p.Gip = p.bf16 ? c.take_bytes((size_t)d * 3 * split_kpad(d) * csz) : nullptr;
  const size_t npad = (size_t)(n + 7) / 8 * 8;   // leading dimension bound of the compact tensors
  // bf16 mode: room for h as hi | lo parts (gated modules)
  p.H = c.take_bytes((size_t)p.chunk * (p.bf16 ? 2 * (size_t)split_kpad(n) : npad) * csz);
  p.E = c.take_bytes((size_t)p.chunk * (p.bf16 ? 2 * (size_t)split_kpad(d) : (size_t)d) * csz);   // hi | lo (gated)
  p.Ac = c.take_bytes((size_t)p.chunk * n * csz);
  p.Zb = p.bf16 ? c.take_bytes((size_t)p.chunk * n * csz) : nullptr;
  p.D = c.take<float>((size_t)p.chunk * npad);
  p.z1 = c.take<float>((size_t)p.chunk * npad);
  p.nblocks = fused_update_grid(p.chunk, n, &p.row_blocks);
  {
    // the form of the update that also writes the next step's operands has its own grid, whose row blocks depend on
    // the chunk's token count: sized for its upper bound
    const int rb2 = fused_update_next_row_cap(n);
    const int64_t nb2 = fused_update_next_max_blocks(n);
    if (nb2 > p.nblocks) p.nblocks = (int)nb2;
    const int pr2 = fused_update_next_partial_rows(rb2);     // (that form leaves several rows of |A| partials per row block)
    if (pr2 > p.row_blocks) p.row_blocks = pr2;
  }
  p.partial = c.take<double>((size_t)p.nblocks * 4 + kSumsqBlocks);
  p.Eo = c.take<float>((size_t)p.chunk * d);
  p.W2fb = p.bf16 ? c.take_bytes((size_t)n * d * csz) : nullptr;
  p.absA_part = c.take<double>((size_t)p.row_blocks * n);
  p.score_scratch = c.take<double>(std::max((size_t)score_row_blocks(d, n) * n * 2 + 16, wanda_scratch_doubles(d, n)));
  p.bytes = align_up(c.off, 256);
  p.z1_all = ws ? reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(ws) + p.bytes) : nullptr;   // optional tail
  return p;
}

size_t overlap_bytes(int64_t N, int64_t k) { return (size_t)N * (size_t)((k + 7) / 8 * 8) * sizeof(float); }

struct InitPlan {
  int64_t chunk;
  bool bf16;
  void *W10b, *W20b, *Wg0b, *Ac, *Zb;   // Wg0b: hi | lo split of the gate weights (gated modules)
  double* absA_part;
  int row_blocks;
  size_t bytes;
};

InitPlan plan_init(void* ws, int64_t d, int64_t n, int64_t N, int64_t chunk, int32_t cdt) {
  InitPlan p;
  p.chunk = chunk > 0 ? chunk : kDefaultChunk;
  if (p.chunk > N) p.chunk = N;
  if (p.chunk < 1) p.chunk = 1;
  p.bf16 = cdt == SP_BF16;
  const size_t csz = p.bf16 ? 2 : 4;
  Carver c(ws);
  p.W10b = p.bf16 ? c.take_bytes((size_t)n * 2 * split_kpad(d) * csz) : nullptr;  // hi | lo split of W1_0
  p.W20b = p.bf16 ? c.take_bytes((size_t)n * d * csz) : nullptr;
  p.Wg0b = p.bf16 ? c.take_bytes((size_t)n * 2 * split_kpad(d) * csz) : nullptr;
  p.Ac = c.take_bytes((size_t)p.chunk * n * csz);
  p.Zb = p.bf16 ? c.take_bytes((size_t)p.chunk * n * csz) : nullptr;
  fused_update_grid(p.chunk, n, &p.row_blocks);
  p.absA_part = c.take<double>((size_t)p.row_blocks * n);
  p.bytes = align_up(c.off, 256);
  return p;
}

size_t ridge_ws_bytes(int64_t m, int64_t n, bool precise) {
  Carver c(nullptr);
  carve_solve(c, n, m, precise ? 8 : 4);
  return align_up(c.off, 256);
}

}  // namespace

extern "C" {

int32_t sp_version(void) { return 100; }

size_t sp_admm_overlap_bytes(int64_t N, int64_t k_keep) { return (N > 0 && k_keep > 0) ? overlap_bytes(N, k_keep) : 0; }

const char* sp_status_string(int32_t s) {
  switch (s) {
    case SP_OK: return "ok";
    case SP_ERR_INVALID_ARG: return "invalid argument";
    case SP_ERR_SHAPE: return "shape mismatch";
    case SP_ERR_DTYPE: return "unsupported dtype";
    case SP_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case SP_ERR_WORKSPACE: return "workspace too small";
    case SP_ERR_NOT_SPD: return "matrix not positive definite";
    case SP_ERR_TIMEOUT: return "bounded device wait ran out";
    case SP_ERR_CUDA: return "CUDA runtime error";
    case SP_ERR_UNSUPPORTED: return "unsupported configuration";
    case SP_ERR_STATIC_LIMIT: return "size exceeds the limit of the built-in static scratch";
    default: return "unknown status";
  }
}

size_t sp_workspace_bytes(int32_t op, int64_t d, int64_t n, int64_t N, int64_t token_chunk, int32_t dtype) {
  switch (op) {
    case SP_WS_GRAM: {
      // d = channels C, N = tokens T
      const int rb = column_stats_row_blocks(N > 0 ? N : 1, d > 0 ? d : 1);
      return align_up((size_t)rb * (size_t)(d > 0 ? d : 1) * 2 * sizeof(double), 256) + 256;
    }
    case SP_WS_ADMM_STEP: return plan_admm(nullptr, d, n, N, token_chunk, dtype).bytes + 256;
    case SP_WS_FFN_INIT: return plan_init(nullptr, d, n, N, token_chunk, dtype).bytes + 256;
    case SP_WS_SCORES: {
      // d = number of columns (n_units * group), N = tokens (LEMMA1) or weight rows (WANDA)
      const int64_t cols = d > 0 ? d : 1;
      const int rb = score_row_blocks(N > 0 ? N : 1, cols);
      const size_t lemma = (size_t)rb * cols * 2 + (size_t)cols * 4 + 16;
      return align_up(std::max(lemma, wanda_scratch_doubles(N > 0 ? N : 1, cols)) * sizeof(double), 256) + 256;
    }
    case SP_WS_APPLY_MASK: return 256;
    case SP_WS_LINEAR_REFIT: return ridge_ws_bytes(d, n, dtype == SP_F64) + align_up((size_t)(n > 0 ? n : 1) * 4, 256) + 512;
    case SP_WS_RIDGE_SOLVE: return ridge_ws_bytes(d, n, dtype == SP_F64) + 256;
    case SP_WS_GEMM: return 256;
    case SP_WS_INPUT_INVERSE:
      return ridge_ws_bytes(d, d, true) + align_up((size_t)(d > 0 ? d : 1) * (size_t)(d > 0 ? d : 1) * 4, 256) + 512;
    case SP_WS_WEIGHT_STATS: return align_up((size_t)(148 * 8 + (d > 0 ? d : 1)) * 3 * sizeof(double), 256) + 256;
    default: return 0;
  }
}

sp_status sp_gemm(int32_t transA, int32_t transB, int64_t M, int64_t N, int64_t K, double alpha, const sp_mat* A,
                  const sp_mat* B, double beta, const sp_mat* C, int32_t lower_only, int32_t use_tensor_cores,
                  int32_t* status_dev, void* stream) {
  if (!A || !B || !C || !A->ptr || !B->ptr || !C->ptr) return SP_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0) return SP_ERR_SHAPE;
  // op(A) is M x K: stored [M,K] when !transA (K-major), [K,M] when transA.
  // op(B) is K x N: stored [K,N] when !transB (N contiguous), [N,K] when transB (K-major).
  const bool a_kmajor = !transA, b_kmajor = transB != 0;
  if (A->ld < (a_kmajor ? K : M) || B->ld < (b_kmajor ? K : N) || C->ld < N) return SP_ERR_SHAPE;
  MatRef a{A->ptr, A->dtype, A->ld}, b{B->ptr, B->dtype, B->ld}, c{C->ptr, C->dtype, C->ld};
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (use_tensor_cores) {
    if (A->dtype != SP_BF16 || B->dtype != SP_BF16 || C->dtype == SP_F64 || K <= 0) return SP_ERR_UNSUPPORTED;
    TcOperand ta{A->ptr, A->ld, a_kmajor}, tb{B->ptr, B->ld, b_kmajor};
    if (!gemm_tc_supported(M, N, K, ta, tb)) return SP_ERR_UNSUPPORTED;
    if (M == 0 || N == 0) return SP_OK;
    return gemm_tc(M, N, K, (float)alpha, ta, tb, (float)beta, Operand{c.ptr, c.dtype, c.ld, 1},
                   OutOperand{const_cast<void*>(c.ptr), c.dtype, c.ld}, lower_only != 0, status_dev, s);
  }
  const bool acc64 = !(A->dtype == SP_BF16 && B->dtype == SP_BF16);
  return contract(M, N, K, alpha, a, a_kmajor, b, b_kmajor, beta, c, c, lower_only != 0, acc64, false, status_dev, s);
}

sp_status sp_symmetrize(float* G, int64_t n, int64_t ldg, void* stream) {
  if (!G) return SP_ERR_INVALID_ARG;
  if (n < 0 || ldg < n) return SP_ERR_SHAPE;
  CU(symmetrize_lower(G, n, ldg, reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

sp_status sp_gram_accumulate(const sp_mat* Xc, const sp_mat* Yc, float* G, int64_t ldg, float* R, int64_t ldr,
                             double* rowstats, int32_t* status_dev, void* ws, size_t ws_bytes, void* stream) {
  if (!Xc || !G) return SP_ERR_INVALID_ARG;
  if (!valid_act_dtype(Xc->dtype)) return SP_ERR_DTYPE;
  const int64_t T = Xc->rows, C = Xc->cols;
  if (T < 0 || C < 0 || Xc->ld < C || ldg < C) return SP_ERR_SHAPE;
  if (!Xc->ptr && T * C > 0) return SP_ERR_INVALID_ARG;   // an empty chunk may carry a null pointer
  if (Yc) {
    if ((!Yc->ptr && T * Yc->cols > 0) || !R) return SP_ERR_INVALID_ARG;
    if (Yc->dtype != Xc->dtype) return SP_ERR_DTYPE;
    if (Yc->rows != T || Yc->ld < Yc->cols || ldr < C) return SP_ERR_SHAPE;
  }
  if (rowstats && (!ws || ws_bytes < sp_workspace_bytes(SP_WS_GRAM, C, 0, T, 0, Xc->dtype))) return SP_ERR_WORKSPACE;
  if (rowstats && misaligned(ws, 8)) return SP_ERR_ALIGNMENT;
  if (T == 0 || C == 0) return SP_OK;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const bool bf16 = Xc->dtype == SP_BF16;
  MatRef x{Xc->ptr, Xc->dtype, Xc->ld};
  MatRef g{G, SP_F32, ldg};
  SPCHK(contract(C, C, T, 1.0, x, false, x, false, 1.0, g, g, true, !bf16, bf16, status_dev, s));
  if (Yc && Yc->cols > 0) {
    MatRef y{Yc->ptr, Yc->dtype, Yc->ld};
    MatRef r{R, SP_F32, ldr};
    SPCHK(contract(Yc->cols, C, T, 1.0, y, false, x, false, 1.0, r, r, false, !bf16, bf16, status_dev, s));
  }
  if (rowstats) CU(column_stats(Xc->ptr, Xc->dtype, Xc->ld, T, C, rowstats, reinterpret_cast<double*>(ws), s));
  return SP_OK;
}

sp_status sp_ridge_solve(const float* R, int64_t ldr, const float* G, int64_t ldg, int64_t m, int64_t n, double rho,
                         int32_t rho_relative, int32_t precise, float* W, int64_t ldw, int32_t* status_dev, void* ws,
                         size_t ws_bytes, void* stream) {
  if (!R || !G || !W) return SP_ERR_INVALID_ARG;
  if (m < 0 || n < 0 || ldr < n || ldg < n || ldw < n) return SP_ERR_SHAPE;
  if (m == 0 || n == 0) return SP_OK;
  if (!ws || ws_bytes < ridge_ws_bytes(m, n, precise != 0)) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  Carver c(ws);
  SolveBufs b = carve_solve(c, n, m, precise ? 8 : 4);
  CU(effective_ridge(G, ldg, n, rho, rho_relative, b.rho, s));
  if (precise) return ridge_core<double>(R, ldr, G, ldg, m, n, nullptr, n, b.rho, W, ldw, b, status_dev, s);
  SideStream* side = side_stream();
  return ridge_core<float>(R, ldr, G, ldg, m, n, nullptr, n, b.rho, W, ldw, b, status_dev, s,
                           side ? &side->assist_main : nullptr);
}

sp_status sp_linear_refit(const float* R, int64_t ldr, const float* G, int64_t ldg, int64_t m, int64_t n_units,
                          int32_t group, const uint8_t* mask, int64_t k_keep, double rho, int32_t rho_relative,
                          int32_t precise, float* W, int64_t ldw, int32_t* status_dev, void* ws, size_t ws_bytes,
                          void* stream) {
  if (!R || !G || !W || !mask) return SP_ERR_INVALID_ARG;
  if (group < 1 || n_units < 0 || m < 0 || k_keep < 0 || k_keep > n_units) return SP_ERR_SHAPE;
  const int64_t n = n_units * group;
  if (ldr < n || ldg < n || ldw < n) return SP_ERR_SHAPE;
  if (m == 0 || n == 0) return SP_OK;
  // workspace: solve buffers for the full size + the unit index list
  const size_t need = ridge_ws_bytes(m, n, precise != 0) + align_up((size_t)n_units * 4, 256);
  if (!ws || ws_bytes < need) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  Carver c(ws);
  SolveBufs b = carve_solve(c, n, m, precise ? 8 : 4);
  int32_t* unit_idx = c.take<int32_t>((size_t)n_units);
  CU(effective_ridge(G, ldg, n, rho, rho_relative, b.rho, s));     // the ridge of the full system
  CU(mask_to_index(mask, n_units, unit_idx, s));
  const int64_t k = k_keep * group;
  if (k > 0) {
    count_launch();
    expand_group_index_kernel<<<(unsigned)ceil_div(k, 256), 256, 0, s>>>(unit_idx, k_keep, group, b.idx);
    CU(cudaGetLastError());
  }
  if (precise) return ridge_core<double>(R, ldr, G, ldg, m, n, b.idx, k, b.rho, W, ldw, b, status_dev, s);
  SideStream* side = side_stream();
  return ridge_core<float>(R, ldr, G, ldg, m, n, b.idx, k, b.rho, W, ldw, b, status_dev, s,
                           side ? &side->assist_main : nullptr);
}

sp_status sp_struct_scores(int32_t kind, int32_t group, const sp_score_inputs* in, int64_t n_units, float* scores,
                           double* layer_importance, double* relaxed_mask, double r_layer, void* ws, size_t ws_bytes,
                           void* stream) {
  if (!in || !scores) return SP_ERR_INVALID_ARG;
  if (group < 1 || n_units < 1) return SP_ERR_SHAPE;
  const int64_t cols = n_units * group;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (kind == SP_SCORE_WANDA_L2 || kind == SP_SCORE_WANDA_L1) {
    if (!in->W.ptr) return SP_ERR_INVALID_ARG;
    if (in->W.dtype != SP_F32) return SP_ERR_DTYPE;
    if (in->W.cols != cols || in->W.ld < cols || in->W.rows < 1) return SP_ERR_SHAPE;
    if (kind == SP_SCORE_WANDA_L2 && (!in->colsq || in->colsq_stride < 1)) return SP_ERR_INVALID_ARG;
    if (kind == SP_SCORE_WANDA_L1 && !in->colabs) return SP_ERR_INVALID_ARG;
    if (relaxed_mask) return SP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < sp_workspace_bytes(SP_WS_SCORES, cols, 0, in->W.rows, 0, SP_F32)) return SP_ERR_WORKSPACE;
    if (misaligned(ws, 8)) return SP_ERR_ALIGNMENT;
    CU(wanda_scores(kind, group, reinterpret_cast<const float*>(in->W.ptr), in->W.rows, in->W.ld, in->colsq,
                    in->colsq_stride, in->colabs, in->inv_tokens, n_units, scores, layer_importance,
                    reinterpret_cast<double*>(ws), s));
    return SP_OK;
  }
  if (kind == SP_SCORE_LEMMA1) {
    const sp_mat* ms[4] = {&in->b, &in->c, &in->dd, &in->t};
    const int64_t N = in->b.rows;
    for (const sp_mat* m : ms) {
      if (!m->ptr) return SP_ERR_INVALID_ARG;
      if (!valid_act_dtype(m->dtype)) return SP_ERR_DTYPE;
      if (m->rows != N || m->cols != cols || m->ld < cols) return SP_ERR_SHAPE;
    }
    if (N < 1) return SP_ERR_SHAPE;
    if (!ws || ws_bytes < sp_workspace_bytes(SP_WS_SCORES, cols, 0, N, 0, SP_F32)) return SP_ERR_WORKSPACE;
    if (misaligned(ws, 8)) return SP_ERR_ALIGNMENT;
    CU(lemma1_scores_stream(in->b, in->c, in->dd, in->t, group, n_units, scores, layer_importance, relaxed_mask,
                            r_layer, reinterpret_cast<double*>(ws), s));
    return SP_OK;
  }
  return SP_ERR_UNSUPPORTED;
}

sp_status sp_allocate_sparsity(const double* I, const int64_t* n_units, int32_t L, double rbar, double T, int32_t mode,
                               double clip_hi, double* r_out, int64_t* k_keep_out, void* stream) {
  if (!I || !n_units || !r_out || !k_keep_out) return SP_ERR_INVALID_ARG;
  if (L < 1 || L > 65536) return SP_ERR_SHAPE;
  if (!(T > 0.0) || !(rbar >= 0.0 && rbar <= 1.0) || !(clip_hi > 0.0 && clip_hi <= 1.0)) return SP_ERR_INVALID_ARG;
  if (mode != SP_ALLOC_SOFTMAX && mode != SP_ALLOC_INVERSE && mode != SP_ALLOC_UNIFORM) return SP_ERR_UNSUPPORTED;
  CU(allocate_sparsity(I, n_units, L, rbar, T, mode, clip_hi, r_out, k_keep_out,
                       reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

sp_status sp_allocate_sparsity_grid(const double* I, const int64_t* n_units, int32_t L, double rbar, const double* T_list,
                                    int32_t n_T, int32_t T_relative, int32_t mode, double clip_hi, double* r_out,
                                    int64_t* k_keep_out, void* stream) {
  if (!I || !n_units || !T_list || !r_out || !k_keep_out) return SP_ERR_INVALID_ARG;
  if (L < 1 || L > 65536 || n_T < 1 || n_T > 65535) return SP_ERR_SHAPE;
  if (!(rbar >= 0.0 && rbar <= 1.0) || !(clip_hi > 0.0 && clip_hi <= 1.0)) return SP_ERR_INVALID_ARG;
  if (mode != SP_ALLOC_SOFTMAX && mode != SP_ALLOC_INVERSE && mode != SP_ALLOC_UNIFORM) return SP_ERR_UNSUPPORTED;
  CU(allocate_sparsity_grid(I, n_units, L, rbar, T_list, n_T, T_relative != 0, mode, clip_hi, r_out, k_keep_out,
                            reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

size_t sp_apply_mask_global_bytes(int64_t n_units, int32_t L) {
  if (n_units < 0 || L < 0) return 0;
  return global_select_scratch_bytes(n_units * (int64_t)L, L) + 256;
}

sp_status sp_apply_mask_global(const float* scores, int64_t ld_scores, int64_t n_units, int32_t L, double keep_fraction,
                               int64_t min_keep, uint8_t* mask_out, int64_t ld_mask, float* tau_out,
                               int64_t* kept_out, void* ws, size_t ws_bytes, void* stream) {
  if (!scores || !mask_out || !kept_out) return SP_ERR_INVALID_ARG;
  if (n_units < 0 || L < 0 || ld_scores < n_units || ld_mask < n_units || min_keep < 0) return SP_ERR_SHAPE;
  if (!(keep_fraction >= 0.0 && keep_fraction <= 1.0)) return SP_ERR_INVALID_ARG;
  if (n_units == 0 || L == 0) return SP_OK;
  if (!ws || ws_bytes < sp_apply_mask_global_bytes(n_units, L)) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  // K = floor(r n L) of Algorithm 3; the small offset keeps products like 0.6 * 5 from falling below their integer
  const int64_t K = (int64_t)floor(keep_fraction * (double)n_units * (double)L + 1e-9);
  CU(global_select(scores, ld_scores, n_units, L, K, min_keep, mask_out, ld_mask, tau_out, kept_out, ws,
                   reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

__global__ void objective_accumulate_kernel(const sp_step_report* rep, double beta, double* loss, int accumulate) {
  const double v = rep->res_out + beta * rep->res_act + rep->res_in;
  loss[0] = accumulate ? loss[0] + v : v;
}

sp_status sp_objective_accumulate(const sp_step_report* rep_dev, double beta, double* loss_dev, int32_t accumulate,
                                  void* stream) {
  if (!rep_dev || !loss_dev) return SP_ERR_INVALID_ARG;
  count_launch();
  objective_accumulate_kernel<<<1, 1, 0, reinterpret_cast<cudaStream_t>(stream)>>>(rep_dev, beta, loss_dev, accumulate);
  CU(cudaGetLastError());
  return SP_OK;
}

sp_status sp_apply_mask(const float* scores, int64_t n_units, int64_t k_keep, int32_t group, uint8_t* mask_out,
                        float* tau_out, int32_t* kept_idx_out, const sp_mat* W_rows, const sp_mat* W_cols, void* ws,
                        size_t ws_bytes, void* stream) {
  (void)ws; (void)ws_bytes;
  if (!scores || !mask_out) return SP_ERR_INVALID_ARG;
  if (n_units < 0 || n_units > 0x7fffffff || group < 1 || k_keep < 0 || k_keep > n_units) return SP_ERR_SHAPE;
  if (W_rows) {
    if (!W_rows->ptr) return SP_ERR_INVALID_ARG;
    if (W_rows->dtype != SP_F32) return SP_ERR_DTYPE;
    if (W_rows->rows != n_units * group || W_rows->ld < W_rows->cols) return SP_ERR_SHAPE;
  }
  if (W_cols) {
    if (!W_cols->ptr) return SP_ERR_INVALID_ARG;
    if (W_cols->dtype != SP_F32) return SP_ERR_DTYPE;
    if (W_cols->cols != n_units * group || W_cols->ld < W_cols->cols) return SP_ERR_SHAPE;
  }
  if (n_units == 0) return SP_OK;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  CU(topk_select(scores, n_units, k_keep, mask_out, tau_out, kept_idx_out, s));
  CU(zero_pruned(mask_out, group, W_rows ? reinterpret_cast<float*>(W_rows->ptr) : nullptr,
                 W_rows ? W_rows->rows : 0, W_rows ? W_rows->cols : 0, W_rows ? W_rows->ld : 0,
                 W_cols ? reinterpret_cast<float*>(W_cols->ptr) : nullptr, W_cols ? W_cols->rows : 0,
                 W_cols ? W_cols->cols : 0, W_cols ? W_cols->ld : 0, s));
  return SP_OK;
}

sp_status sp_apply_mask_batched(const float* scores, int64_t ld_scores, int64_t n_units, int32_t L,
                                const int64_t* k_keep, uint8_t* mask_out, int64_t ld_mask, float* tau_out,
                                int32_t* kept_idx_out, int64_t ld_idx, void* stream) {
  if (!scores || !k_keep || !mask_out) return SP_ERR_INVALID_ARG;
  if (n_units < 0 || n_units > 0x7fffffff || L < 0) return SP_ERR_SHAPE;
  if (ld_scores < n_units || ld_mask < n_units || (kept_idx_out && ld_idx < n_units)) return SP_ERR_SHAPE;
  if (n_units == 0 || L == 0) return SP_OK;
  CU(topk_select_batched(scores, ld_scores, n_units, L, 0, k_keep, mask_out, ld_mask, tau_out, kept_idx_out, ld_idx,
                         reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

sp_status sp_weight_stats(const sp_mat* W, int32_t axis, int64_t group, int32_t accumulate, double* stats, void* ws,
                          size_t ws_bytes, void* stream) {
  if (!W || !W->ptr || !stats || (axis != 0 && axis != 1)) return SP_ERR_INVALID_ARG;
  if (W->dtype != SP_F32 && W->dtype != SP_BF16) return SP_ERR_DTYPE;
  if (W->rows < 0 || W->cols < 0 || W->ld < W->cols || group < 0) return SP_ERR_SHAPE;
  if (group > 0 && (axis == 0 ? W->rows % group : W->cols % group) != 0) return SP_ERR_SHAPE;
  if (W->rows == 0 || W->cols == 0) return SP_OK;
  const int64_t n_blocks = group > 0 ? (axis == 0 ? W->rows / group : W->cols / group) : 1;
  if (!ws || ws_bytes < sp_workspace_bytes(SP_WS_WEIGHT_STATS, n_blocks, 0, 0, 0, 0)) return SP_ERR_WORKSPACE;
  CU(weight_stats(W->ptr, W->dtype, W->ld, W->rows, W->cols, axis, group, accumulate != 0, stats,
                  reinterpret_cast<double*>(align_up(reinterpret_cast<uintptr_t>(ws), 256)),
                  reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

sp_status sp_distribute_importance(const double* head_stats, int32_t n_heads, const double* fc_stats, int32_t n_fc,
                                   int32_t L, double rho, double gamma, double* I_attn, double* I_mlp, void* stream) {
  if (L < 0 || n_heads < 0 || n_fc < 0) return SP_ERR_SHAPE;
  if ((head_stats && !I_attn) || (fc_stats && !I_mlp) || (!head_stats && !fc_stats)) return SP_ERR_INVALID_ARG;
  CU(distribute_importance(head_stats, n_heads, fc_stats, n_fc, L, rho, gamma, I_attn, I_mlp,
                           reinterpret_cast<cudaStream_t>(stream)));
  return SP_OK;
}

static sp_status check_module(const sp_ffn_module* m, const sp_ffn_state* st, bool need_w0) {
  if (!m || !st) return SP_ERR_INVALID_ARG;
  if (m->d < 1 || m->n < 1 || m->N < 1) return SP_ERR_SHAPE;
  if (m->act != SP_ACT_RELU && m->act != SP_ACT_SWIGLU) return SP_ERR_UNSUPPORTED;
  if (m->act == SP_ACT_SWIGLU) {
    if (!st->Gate) return SP_ERR_INVALID_ARG;
    if (need_w0) {
      if (!m->Wg_0.ptr) return SP_ERR_INVALID_ARG;
      if (m->Wg_0.dtype != SP_F32) return SP_ERR_DTYPE;
      if (m->Wg_0.rows != m->n || m->Wg_0.cols != m->d || m->Wg_0.ld < m->d) return SP_ERR_SHAPE;
    }
  }
  if (!m->X.ptr || !m->Ypre.ptr) return SP_ERR_INVALID_ARG;
  if (!valid_act_dtype(m->X.dtype) || m->Ypre.dtype != m->X.dtype) return SP_ERR_DTYPE;
  if (m->X.rows != m->N || m->X.cols != m->d || m->X.ld < m->d) return SP_ERR_SHAPE;
  if (m->Ypre.rows != m->N || m->Ypre.cols != m->d || m->Ypre.ld < m->d) return SP_ERR_SHAPE;
  if (need_w0) {
    if (!m->W1_0.ptr || !m->W2_0.ptr) return SP_ERR_INVALID_ARG;
    if (m->W1_0.dtype != SP_F32 || m->W2_0.dtype != SP_F32) return SP_ERR_DTYPE;
    if (m->W1_0.rows != m->n || m->W1_0.cols != m->d || m->W1_0.ld < m->d) return SP_ERR_SHAPE;
    if (m->W2_0.rows != m->d || m->W2_0.cols != m->n || m->W2_0.ld < m->n) return SP_ERR_SHAPE;
  }
  if (!st->Z || !st->G_X || !st->G_A || !st->R1 || !st->R2 || !st->absA) return SP_ERR_INVALID_ARG;
  return SP_OK;
}

sp_status sp_ffn_init(const sp_ffn_module* m, sp_ffn_state* st, int64_t token_chunk, int32_t* status_dev, void* ws,
                      size_t ws_bytes, void* stream) {
  SPCHK(check_module(m, st, true));
  if (token_chunk < 0) return SP_ERR_INVALID_ARG;
  const int64_t d = m->d, n = m->n, N = m->N;
  const int32_t cdt = m->X.dtype;
  if (!ws || ws_bytes < plan_init(nullptr, d, n, N, token_chunk, cdt).bytes) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256) || misaligned(st->Z, 16) || misaligned(st->U, 16) || misaligned(st->Gate, 16) ||
      misaligned(m->X.ptr, 16) || misaligned(m->Ypre.ptr, 16))
    return SP_ERR_ALIGNMENT;
  InitPlan p = plan_init(ws, d, n, N, token_chunk, cdt);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const bool bf16 = p.bf16;
  if (st->decay_tag != nullptr) CU(decay_tag_set(st->decay_tag, 0, 0.f, false, 0, 0, s));   // Z is rewritten
  const bool acc64 = !bf16;
  const bool gated = m->act == SP_ACT_SWIGLU;
  MatRef w10{m->W1_0.ptr, SP_F32, m->W1_0.ld}, w20{m->W2_0.ptr, SP_F32, m->W2_0.ld};
  MatRef wg0{gated ? m->Wg_0.ptr : nullptr, SP_F32, gated ? m->Wg_0.ld : 0};
  if (bf16) {
    if (gated)
      CU(split_bf16(reinterpret_cast<const float*>(m->Wg_0.ptr), m->Wg_0.ld, nullptr, n, d, split_kpad(d), p.Wg0b, s));
    CU(split_bf16(reinterpret_cast<const float*>(m->W1_0.ptr), m->W1_0.ld, nullptr, n, d, split_kpad(d), p.W10b, s));
    CU(convert_matrix(m->W2_0.ptr, SP_F32, m->W2_0.ld, p.W20b, SP_BF16, n, d, n, s));
    w20 = MatRef{p.W20b, SP_BF16, n};
  }
  if (st->U) CU(cudaMemsetAsync(st->U, 0, (size_t)N * n * sizeof(float), s));
  const size_t esz = bf16 ? 2 : 4;
  MatRef gx{st->G_X, SP_F32, d}, ga{st->G_A, SP_F32, n}, r1{st->R1, SP_F32, d}, r2{st->R2, SP_F32, n};
  for (int64_t t0 = 0, ci = 0; t0 < N; t0 += p.chunk, ++ci) {
    const int64_t Tc = (N - t0 < p.chunk) ? N - t0 : p.chunk;
    const double acc = ci > 0 ? 1.0 : 0.0;
    MatRef xc{reinterpret_cast<const uint8_t*>(m->X.ptr) + (size_t)t0 * m->X.ld * esz, cdt, m->X.ld};
    MatRef yc{reinterpret_cast<uint8_t*>(m->Ypre.ptr) + (size_t)t0 * m->Ypre.ld * esz, cdt, m->Ypre.ld};
    float* Zc = st->Z + (size_t)t0 * n;
    MatRef zc{Zc, SP_F32, n};
    MatRef ac{p.Ac, cdt, n};
    MatRef zb = bf16 ? MatRef{p.Zb, cdt, n} : zc;
    // z^pre = X W1_0^T
    if (bf16) SPCHK(contract_split_weights(Tc, n, d, xc, p.W10b, w10, zc, status_dev, s));
    else SPCHK(contract(Tc, n, d, 1.0, xc, true, w10, true, 0.0, zc, zc, false, acc64, false, status_dev, s));
    float* Gc = gated ? st->Gate + (size_t)t0 * n : nullptr;
    if (gated) {   // gate pre-activation X Wg_0^T into the gate buffer; the activation kernel turns it into SiLU
      MatRef gc{Gc, SP_F32, n};
      if (bf16) SPCHK(contract_split_weights(Tc, n, d, xc, p.Wg0b, wg0, gc, status_dev, s));
      else SPCHK(contract(Tc, n, d, 1.0, xc, true, wg0, true, 0.0, gc, gc, false, acc64, false, status_dev, s));
    }
    int rb;
    fused_update_grid(Tc, n, &rb);
    CU(launch_init_act(Zc, Gc, p.Ac, p.Zb, cdt, Tc, n, p.absA_part, rb, s));
    CU(reduce_col_partials(p.absA_part, rb, n, st->absA, ci > 0, s));
    // Ypre = a^pre W2_0^T
    SPCHK(contract(Tc, d, n, 1.0, ac, true, w20, true, 0.0, yc, yc, false, acc64, bf16, status_dev, s));
    // accumulators
    SPCHK(contract(d, d, Tc, 1.0, xc, false, xc, false, acc, gx, gx, true, acc64, bf16, status_dev, s));
    SPCHK(contract(n, n, Tc, 1.0, ac, false, ac, false, acc, ga, ga, true, acc64, bf16, status_dev, s));
    SPCHK(contract(n, d, Tc, 1.0, zb, false, xc, false, acc, r1, r1, false, acc64, bf16, status_dev, s));
    SPCHK(contract(d, n, Tc, 1.0, yc, false, ac, false, acc, r2, r2, false, acc64, bf16, status_dev, s));
  }
  CU(symmetrize_lower(st->G_X, d, d, s));
  CU(symmetrize_lower(st->G_A, n, n, s));
  return SP_OK;
}

sp_status sp_ffn_cache_input_inverse(const sp_ffn_module* m, sp_ffn_state* st, double rho, int32_t rho_relative,
                                     int32_t* status_dev, void* ws, size_t ws_bytes, void* stream) {
  if (!m || !st || !st->G_X || !st->G_X_inv || !(rho >= 0.0)) return SP_ERR_INVALID_ARG;
  const int64_t d = m->d;
  if (d < 1) return SP_ERR_SHAPE;
  if (!ws || ws_bytes < sp_workspace_bytes(SP_WS_INPUT_INVERSE, d, 0, 0, 0, 0)) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  Carver c(ws);
  SolveBufs b = carve_solve(c, d, d, 8);
  float* eye = c.take<float>((size_t)d * d);
  CU(set_identity(eye, d, d, s));
  CU(effective_ridge(st->G_X, d, d, rho, rho_relative, b.rho, s));
  return ridge_core<double>(eye, d, st->G_X, d, d, d, nullptr, d, b.rho, st->G_X_inv, d, b, status_dev, s);
}

// One step, or (scores_only) its first two parts: the unrestricted recovery the scores read, and the scores.
static sp_status admm_step_impl(const sp_ffn_module* m, sp_ffn_state* st, const sp_admm_params* prm, sp_step_report* rep_dev,
                         int32_t* status_dev, void* ws, size_t ws_bytes, void* stream, bool scores_only) {
  if (!prm) return SP_ERR_INVALID_ARG;
  SPCHK(check_module(m, st, prm->score_kind == SP_SCORE_LEMMA1));
  if (!st->W1 || !st->W2 || !st->scores || !st->mask || !st->importance) return SP_ERR_INVALID_ARG;
  if (prm->dual_mode && !st->U) return SP_ERR_INVALID_ARG;
  const int64_t d = m->d, n = m->n, N = m->N;
  if (scores_only && prm->skip_scores) return SP_ERR_INVALID_ARG;
  if (!scores_only && (prm->k_keep < 1 || prm->k_keep > n)) return SP_ERR_SHAPE;
  if (prm->score_kind == SP_SCORE_LEMMA1 && m->W1_0.ld != d) return SP_ERR_SHAPE;
  if (!(prm->alpha > 0.0) || !(prm->beta > 0.0) || !(prm->rho >= 0.0) || prm->token_chunk < 0) return SP_ERR_INVALID_ARG;
  if (prm->z_rule != SP_Z_PAPER && prm->z_rule != SP_Z_EXACT) return SP_ERR_UNSUPPORTED;
  if (prm->score_kind < SP_SCORE_WANDA_L2 || prm->score_kind > SP_SCORE_LEMMA1) return SP_ERR_UNSUPPORTED;
  if (m->act == SP_ACT_SWIGLU && prm->score_kind == SP_SCORE_LEMMA1) return SP_ERR_UNSUPPORTED;
  if (prm->skip_scores && (prm->reselect_mask || !prm->refit)) return SP_ERR_INVALID_ARG;
  const int32_t cdt = m->X.dtype;
  if (!ws || ws_bytes < plan_admm(nullptr, d, n, N, prm->token_chunk, cdt).bytes) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256) || misaligned(st->Z, 16) || misaligned(st->U, 16) || misaligned(st->Gate, 16) ||
      misaligned(m->X.ptr, 16) || misaligned(m->Ypre.ptr, 16))
    return SP_ERR_ALIGNMENT;
  AdmmPlan p = plan_admm(ws, d, n, N, prm->token_chunk, cdt);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const bool bf16 = p.bf16;
  const bool acc64 = !bf16;
  const int64_t k = prm->k_keep;
  double* rho1 = p.sb.rho;
  double* rho2 = p.sb.rho + 1;
  double* gam = p.sb.rho + 2;

  // ---- 1. weight recovery W1~ = R1 (G_X + rho1 I)^-1, W2~ = R2 (G_A + rho2 I)^-1
  // The two recoveries are independent; both are chains of short kernels that leave most SMs idle, so the W1 chain
  // runs on the side stream while the caller's stream carries the W2 chain.
  SideStream* side = side_stream();
  cudaStream_t sa = side ? side->stream : s;
  JoinOnExit join_guard{side, s};
  // Reuse of the factorisation for the recovery on the kept support (tensor-core path): the unrestricted system is
  // solved with the channels that the mask kept so far in front.  The leading block of that factor is the factor of
  // the restricted system of those channels, and the leading columns of the forward-substituted right-hand sides are
  // its forward substitution.  When the new top-k selects the same channels (a device flag, no host round trip), the
  // restricted recovery is one backward sweep; otherwise the restricted system is factorised as usual.  The kernels
  // of both branches are always queued and return at once when their branch is not taken.
  const bool skip_scores = prm->skip_scores != 0;   // fixed mask: W2~ and the scores serve nothing
  const int64_t k_lead = chol_tc_pad(k);
  const bool reuse = bf16 && !skip_scores && !scores_only && prm->refit && k < n && k_lead <= n;
  const LeadSave lead{p.W2cf, k, k_lead};     // W2cf is free until the operands of the token pass are built
  if (reuse) CU(mask_to_perm(st->mask, n, p.perm, p.reuse_flags + 2, s));
  if (side) {
    CU(cudaEventRecord(side->fork, s));
    CU(cudaStreamWaitEvent(sa, side->fork, 0));
  }
  // The long chain (W2, on the caller's stream) is queued first: queuing the W1 chain takes the host more than half a
  // millisecond, during which the caller's stream would otherwise sit empty.  (Without a side stream both run on
  // the caller's stream and the order does not matter.)
  CU(effective_ridge(st->G_A, n, n, prm->rho, prm->rho_relative, rho2, s));
  if (skip_scores) {
  } else if (bf16) {
    SPCHK(ridge_core<float>(st->R2, n, st->G_A, n, d, n, reuse ? p.perm : nullptr, n, rho2, p.W2t, n, p.sb, status_dev,
                            s, side ? &side->assist_main : nullptr, false, reuse ? &lead : nullptr));
  } else {
    SPCHK(ridge_core<double>(st->R2, n, st->G_A, n, d, n, nullptr, n, rho2, p.W2t, n, p.sb, status_dev, s,
                             side ? &side->assist_main : nullptr));
  }
  const bool need_w1 = !scores_only || prm->score_kind == SP_SCORE_LEMMA1;   // only the Lemma-1 score reads W1~
  if (need_w1) {
    CU(effective_ridge(st->G_X, d, d, prm->rho, prm->rho_relative, rho1, sa));
    if (bf16 && st->G_X_inv) {
      // cached inverse of the constant system: W1~ = R1 Ginv, both operands as three bf16 parts, the six part products
      // of weight >= 2^-16 as K segments (Ginv is symmetric, so its rows serve as the K-major B operand)
      const int64_t dp3 = split_kpad(d);
      CU(split3_bf16(st->R1, d, n, d, dp3, p.R1p, sa));
      CU(split3_bf16(st->G_X_inv, d, d, d, dp3, p.Gip, sa));
      TcOperand ta{p.R1p, 3 * dp3, true}, tb{p.Gip, 3 * dp3, true};
      ta.kext = tb.kext = 3 * dp3;
      TcSegments sg;
      sg.nseg = 6;
      static const int pa[6] = {0, 0, 1, 0, 2, 1}, pb[6] = {0, 1, 0, 2, 0, 1};
      for (int q = 0; q < 6; ++q) {
        sg.a_k[q] = (int32_t)(pa[q] * dp3);
        sg.b_k[q] = (int32_t)(pb[q] * dp3);
      }
      ProfScope prof(PK_SOLVE, 2.0 * (double)n * d * d, 0.0, sa);
      SPCHK(gemm_tc(n, d, d, 1.f, ta, tb, 0.f, Operand{p.W1t, SP_F32, d, 1}, OutOperand{p.W1t, SP_F32, d}, false,
                    status_dev, sa, &sg, 2.0 * (double)n * d * d));
    } else if (bf16) SPCHK(ridge_core<float>(st->R1, d, st->G_X, d, n, d, nullptr, d, rho1, p.W1t, d, p.sbA, status_dev, sa,
                                      side ? &side->assist_side : nullptr));
    else SPCHK(ridge_core<double>(st->R1, d, st->G_X, d, n, d, nullptr, d, rho1, p.W1t, d, p.sbA, status_dev, sa,
                                      side ? &side->assist_side : nullptr));
  }
  if (side) CU(cudaEventRecord(side->join, sa));
  bool joined = side == nullptr;

  // ---- 2. unit scores and layer importance
  if (skip_scores) {
  } else if (prm->score_kind == SP_SCORE_LEMMA1) {
    if (!joined) { CU(cudaStreamWaitEvent(s, side->join, 0)); joined = true; }   // this score reads W1~
    // b = W1~ X, c = d = t = z^pre = W1_0 X, written through G_X:  T0 = W1_0 G_X
    MatRef w10{m->W1_0.ptr, SP_F32, m->W1_0.ld}, gx{st->G_X, SP_F32, d}, t0{p.T0, SP_F32, d};
    SPCHK(contract(n, d, d, 1.0, w10, true, gx, false, 0.0, t0, t0, false, true, false, status_dev, s));
    CU(lemma1_scores_gram(p.T0, p.W1t, reinterpret_cast<const float*>(m->W1_0.ptr), n, d, st->scores, st->importance,
                          p.score_scratch, s));
  } else {
    CU(wanda_scores(prm->score_kind, 1, p.W2t, d, n, st->G_A, n + 1, st->absA, 1.0 / (double)N, n, st->scores,
                    st->importance, p.score_scratch, s));
  }

  if (scores_only) {
    if (!joined) CU(cudaStreamWaitEvent(s, side->join, 0));
    join_guard.armed = false;
    return SP_OK;
  }

  // ---- 3. top-k mask
  if (prm->reselect_mask) CU(topk_select(st->scores, n, k, st->mask, nullptr, p.sb.idx, s));
  else {
    CU(mask_to_index(st->mask, n, p.sb.idx, s));
    CU(mask_count_check(st->mask, n, k, status_dev, s));     // a given mask must keep exactly k_keep units
  }
  if (reuse) CU(mask_changed(st->mask, p.perm, p.reuse_flags + 2, k, p.reuse_flags, s));

  // ---- 4. masked weights: W1 = diag(M) W1~ ; W2 = recovery on the kept support (or M (.) W2~)
  if (!joined) { CU(cudaStreamWaitEvent(s, side->join, 0)); joined = true; }
  CU(mask_rows_copy(st->mask, p.W1t, d, st->W1, d, n, d, s));
  // z1 = X W1[S, :]^T needs only the mask and W1: when the workspace has room for z1 of all tokens, these products
  // run on the side stream, on a subset of the SMs, while the caller's stream carries the recovery of W2 on the kept
  // support and the operands of the a-update (chains of short kernels that cannot fill the GPU).
  const int64_t kp_ahead = (k + 7) / 8 * 8;
  const bool z1_ahead = bf16 && side != nullptr && ws_bytes >= p.bytes + overlap_bytes(N, k);
  if (z1_ahead) {
    CU(cudaEventRecord(side->fork, s));
    CU(cudaStreamWaitEvent(side->stream, side->fork, 0));
    CU(split_bf16(st->W1, d, p.sb.idx, k, d, split_kpad(d), p.W1b, side->stream));
    const size_t esz_x = 2;
    for (int64_t t0 = 0; t0 < N; t0 += p.chunk) {
      const int64_t Tc = (N - t0 < p.chunk) ? N - t0 : p.chunk;
      MatRef xc{reinterpret_cast<const uint8_t*>(m->X.ptr) + (size_t)t0 * m->X.ld * esz_x, cdt, m->X.ld};
      MatRef z1c{p.z1_all + (size_t)t0 * kp_ahead, SP_F32, kp_ahead};
      SPCHK(contract_split_weights(Tc, k, d, xc, p.W1b, MatRef{nullptr, SP_F32, d}, z1c, status_dev, side->stream,
                                   kZ1AheadPairs));
    }
    CU(cudaEventRecord(side->z1_done, side->stream));
  }
  if (prm->refit) {
    // beside the z1 products the lookahead kernel of the factorisation runs as two launches of independent CTAs: a
    // cluster of 8 would wait for a free group of SMs while the persistent GEMM CTAs hold most of them
    if (reuse) {
      {
        SkipScope skip_if_changed(p.reuse_flags + 0);
        ProfScope prof(PK_SOLVE, 2.0 * (double)d * k_lead * k_lead, 0.0, s);
        SPCHK(potrs_right_tc(lead.Y, d, k_lead, k_lead, p.sb.P, reinterpret_cast<const float*>(p.sb.dinv), p.sb.Xs,
                             status_dev, s, side ? &side->assist_main : nullptr, true,
                             reinterpret_cast<const float*>(p.sb.Gs), n, n));
        CU(scatter_cols<float>(lead.Y, k_lead, p.sb.idx, d, k, n, st->W2, n, s));
      }
      {
        SkipScope skip_if_unchanged(p.reuse_flags + 1);
        SPCHK(ridge_core<float>(st->R2, n, st->G_A, n, d, n, p.sb.idx, k, rho2, st->W2, n, p.sb, status_dev, s,
                                side ? &side->assist_main : nullptr, z1_ahead, nullptr, true));
      }
    } else if (bf16) {
      SPCHK(ridge_core<float>(st->R2, n, st->G_A, n, d, n, p.sb.idx, k, rho2, st->W2, n, p.sb, status_dev, s,
                              side ? &side->assist_main : nullptr, z1_ahead));
    } else {
      SPCHK(ridge_core<double>(st->R2, n, st->G_A, n, d, n, p.sb.idx, k, rho2, st->W2, n, p.sb, status_dev, s,
                               side ? &side->assist_main : nullptr));
    }
  } else {
    CU(cudaMemcpyAsync(st->W2, p.W2t, (size_t)d * n * sizeof(float), cudaMemcpyDeviceToDevice, s));
    CU(zero_pruned(st->mask, 1, nullptr, 0, 0, 0, st->W2, d, n, n, s));
  }

  // ---- 5a. operands of the token pass, all on the kept support S (k channels, compact, ascending channel order):
  //      W1[S, :], W2[:, S], C = gamma I + W2 W2^T (d x d), Qt = W2[:, S]^T C^-1 (k x d)
  const int64_t kp = (k + 7) / 8 * 8;            // leading dimension of the compact [., k] tensors
  const int32_t* idx = p.sb.idx;
  // Gated modules in bf16 mode: E = Ypre - h W2^T is a small difference of large terms (|h| can exceed |E| by two
  // orders of magnitude when gate factors are large), so one bf16 rounding of h and of W2 would dominate the error of
  // the a-update.  Both operands of that product are carried as bf16 hi + lo parts (three K segments: hi.hi, lo.hi,
  // hi.lo), which keeps about 16 bits of each.
  // E itself is then written as hi + lo parts as well and D = E Q^T takes two K segments (E_hi, E_lo against Q).
  const bool split_h = bf16 && m->act == SP_ACT_SWIGLU;
  const int64_t kp64 = split_kpad(k), dp64 = split_kpad(d);
  if (split_h && dp64 != d) CU(cudaMemsetAsync(p.E, 0, (size_t)p.chunk * 2 * dp64 * 2, s));   // padding columns stay zero
  CU(build_group_map(st->mask, n, p.grp_base, p.grp_mask, s));
  CU(gather_cols<float>(st->W2, n, idx, d, k, p.W2cf, kp, s));
  MatRef w1{nullptr, SP_F32, d}, w2{p.W2cf, SP_F32, kp}, qt{p.Qt, SP_F32, d};
  if (bf16) {
    if (!z1_ahead) CU(split_bf16(st->W1, d, idx, k, d, split_kpad(d), p.W1b, s));
    CU(convert_matrix(p.W2cf, SP_F32, kp, p.W2b, SP_BF16, kp, d, k, s));
    w2 = MatRef{p.W2b, SP_BF16, kp};
    if (split_h) CU(split_bf16(p.W2cf, kp, nullptr, d, k, kp64, p.W2sb, s));
  } else {
    CU(gather_rows(st->W1, d, idx, k, d, p.W1c, d, s));
    w1 = MatRef{p.W1c, SP_F32, d};
  }
  {
    MatRef cf{p.Cf, SP_F32, d};
    SPCHK(contract(d, d, k, 1.0, w2, true, w2, true, 0.0, cf, cf, true, acc64, bf16, status_dev, s));
    CU(effective_ridge(nullptr, 0, 1, prm->beta / prm->alpha, 0, gam, s));
    ProfScope prof(PK_SOLVE, (double)d * d * d / 3.0 + 2.0 * (double)k * d * d, 0.0, s);
    if (bf16) {
      float* Gs = reinterpret_cast<float*>(p.sb.Gs);
      float* Rs = Gs + (size_t)d * d;     // right-hand sides below the system matrix: they ride through the factorisation
      CU(load_spd<float>(p.Cf, d, d, gam, Gs, d, s));
      // right-hand sides: the rows of W2[:, S]^T as the tensor-core path sees them (bf16-rounded)
      CU(convert_matrix(p.W2b, SP_BF16, kp, p.W2cf, SP_F32, kp, d, k, s));
      CU(transpose_convert<float>(p.W2cf, kp, d, k, Rs, d, s));
      SPCHK(potrf_lower_tc(Gs, d, d, reinterpret_cast<float*>(p.sb.dinv), p.sb.P, status_dev, s,
                           side ? &side->assist_main : nullptr, k, z1_ahead));
      SPCHK(potrs_right_tc(Rs, k, d, d, p.sb.P, reinterpret_cast<float*>(p.sb.dinv), p.sb.Xs, status_dev, s,
                           side ? &side->assist_main : nullptr, true, Gs, d));
      if (split_h) {
        CU(split_bf16(Rs, d, nullptr, k, d, dp64, p.Qtb, s));      // only the hi part is used (see the D product)
        qt = MatRef{p.Qtb, SP_BF16, 2 * dp64};
      } else {
        CU(convert_matrix(Rs, SP_F32, d, p.Qtb, SP_BF16, d, k, d, s));
        qt = MatRef{p.Qtb, SP_BF16, d};
      }
    } else {
      double* Gs = reinterpret_cast<double*>(p.sb.Gs);
      double* Rs = Gs + (size_t)d * d;
      CU(load_spd<double>(p.Cf, d, d, gam, Gs, d, s));
      CU(potrf_lower<double>(Gs, d, d, reinterpret_cast<double*>(p.sb.dinv), status_dev, s));
      CU(transpose_convert<double>(p.W2cf, kp, d, k, Rs, d, s));
      CU(potrs_right<double>(Rs, k, d, d, Gs, d, reinterpret_cast<double*>(p.sb.dinv), s));
      CU(convert_matrix(Rs, SP_F64, d, p.Qt, SP_F32, d, k, d, s));
    }
  }

  if (rep_dev && prm->compute_objective && bf16) CU(convert_matrix(st->W2, SP_F32, n, p.W2fb, SP_BF16, n, d, n, s));

  // ---- 5b. token pass
  // Pruned channels (ReLU, no dual variable): a = phi(z) and z_new = c max(z, 0) with c = beta / (alpha + beta), so
  // from the second step with an unchanged mask on their rows of A are c times those of the step before.  The
  // accumulators are therefore built in "kept channels first" order in buffers that persist in the state: the kept
  // columns are contracted over the tokens in every step, the pruned x pruned block of G_A and the pruned columns
  // of R2 only when the channel order differs from the last token pass; otherwise they are last step's values times
  // c^2 and c (c of the step that wrote them).  The branch is a device flag; both sets of kernels are queued.
  const bool decay = bf16 && !scores_only && m->act == SP_ACT_RELU && !prm->dual_mode && n % 4 == 0 && k < n &&
                     p.chunk % 8 == 0 && !(rep_dev && prm->compute_objective) && st->G_A_perm != nullptr &&
                     st->R2_perm != nullptr && st->decay_tag != nullptr && !misaligned(st->G_A_perm, 16) &&
                     !misaligned(st->R2_perm, 16) && !misaligned(st->decay_tag, 4);
  // R1 the same way (Z of a pruned channel is c times its old value as well).  Its operand then is a bf16 copy of the
  // new Z written TRANSPOSED with the kept channels first, by the fused update itself, which also leaves
  // h = max(Z_new, 0) of the kept channels (transposed as well: chunk by chunk a [k, chunk] block of H_next, the block
  // of the chunk that starts at token t0 at element t0 * H_next_ld) for the next step, whose own gather pass over Z is
  // then skipped while the mask stays: Z is read once and written once per step.
  const int64_t ldh_next = st->H_next_ld;
  const bool decay_z = decay && st->R1_perm != nullptr && st->H_next != nullptr && ldh_next % 8 == 0 && ldh_next >= kp &&
                       N % 8 == 0 && !misaligned(st->R1_perm, 16) && !misaligned(st->H_next, 16);
  int32_t* order_changed = p.reuse_flags + 4;
  int32_t* order_same = p.reuse_flags + 5;
  int32_t* h_ready = p.reuse_flags + 6;
  if (decay) {
    // tag: [1] k of the last pass (-1: none), [2] its c (float bits), [4] row pitch of the h it left, [8..] its order
    int32_t* tag = st->decay_tag;
    CU(mask_changed(st->mask, tag + 8, tag + 1, k, order_changed, s));
    if (decay_z) CU(h_next_ready(order_same, tag, ldh_next, p.chunk, h_ready, s));
    {
      SkipScope unless_same(order_changed);
      CU(scale_block(st->G_A_perm + (size_t)k * n + k, n, n - k, n - k, tag + 2, 2, s));
      CU(scale_block(st->R2_perm + k, n, d, n - k, tag + 2, 1, s));
    }
    CU(mask_to_perm(st->mask, n, tag + 8, tag + 3, s));
    CU(decay_tag_set(tag, k, (float)(prm->beta / (prm->alpha + prm->beta)), true, decay_z ? ldh_next : 0, p.chunk, s));
    if (decay_z) {
      // Z_new = c max(Z, 0) with THIS step's c (A above is max(Z, 0) of the old Z: the c of the step that wrote it);
      // R1_perm and H_next hold the last pass's values only if that pass wrote them
      SkipScope unless_ready(h_ready + 1);
      CU(scale_block(st->R1_perm + (size_t)k * d, d, n - k, d, tag + 2, 1, s));
    }
  } else if (!scores_only && st->decay_tag != nullptr) {
    CU(decay_tag_set(st->decay_tag, 0, 0.f, false, 0, 0, s));    // Z changes without the ordered accumulators being rebuilt
  }
  if (z1_ahead) CU(cudaStreamWaitEvent(s, side->z1_done, 0));
  if (rep_dev) CU(init_report(rep_dev, rho1, rho2, (double)k, reuse ? p.reuse_flags + 1 : nullptr,
                              decay ? order_same : nullptr, s));
  const size_t esz = bf16 ? 2 : 4;
  MatRef ga{st->G_A, SP_F32, n}, r1{st->R1, SP_F32, d}, r2{st->R2, SP_F32, n};
  for (int64_t t0 = 0, ci = 0; t0 < N; t0 += p.chunk, ++ci) {
    const int64_t Tc = (N - t0 < p.chunk) ? N - t0 : p.chunk;
    const double acc = ci > 0 ? 1.0 : 0.0;
    MatRef xc{reinterpret_cast<const uint8_t*>(m->X.ptr) + (size_t)t0 * m->X.ld * esz, cdt, m->X.ld};
    MatRef yc{reinterpret_cast<const uint8_t*>(m->Ypre.ptr) + (size_t)t0 * m->Ypre.ld * esz, cdt, m->Ypre.ld};
    float* Zc = st->Z + (size_t)t0 * n;
    float* Uc = (prm->dual_mode && st->U) ? st->U + (size_t)t0 * n : nullptr;
    MatRef h{p.H, cdt, kp}, e{p.E, cdt, d}, dd{p.D, SP_F32, kp}, z1{p.z1, SP_F32, kp}, ac{p.Ac, cdt, n};
    MatRef zb = bf16 ? MatRef{p.Zb, cdt, n} : MatRef{Zc, SP_F32, n};
    const float* Gc = (m->act == SP_ACT_SWIGLU) ? st->Gate + (size_t)t0 * n : nullptr;
    // E = Ypre - h_S W2[:, S]^T ; D_S = E Qt^T ; z1_S = X W1[S, :]^T
    if (split_h) {
      CU(launch_prep_h(Zc, Uc, Gc, p.H, cdt, Tc, n, 2 * kp64, k, idx, s, kp64));
      TcOperand ta{p.H, 2 * kp64, true}, tb{p.W2sb, 2 * kp64, true};
      ta.kext = tb.kext = 2 * kp64;
      TcSegments sg;
      sg.nseg = 3;
      sg.a_k[1] = (int32_t)kp64;      // lo(h) . hi(W2)
      sg.b_k[2] = (int32_t)kp64;      // hi(h) . lo(W2)
      OutOperand e_out{p.E, cdt, 2 * dp64};
      e_out.lo_off = dp64;
      SPCHK(gemm_tc(Tc, d, k, -1.f, ta, tb, 1.f, Operand{yc.ptr, cdt, yc.ld, 1}, e_out, false, status_dev, s, &sg,
                    2.0 * (double)Tc * d * k));
      // D = E Q^T with E = E_hi + E_lo
      TcOperand da{p.E, 2 * dp64, true}, db{qt.ptr, qt.ld, true};
      da.kext = 2 * dp64;
      db.kext = d;
      TcSegments sd;
      sd.nseg = 2;
      sd.a_k[1] = (int32_t)dp64;
      SPCHK(gemm_tc(Tc, k, d, 1.f, da, db, 0.f, Operand{p.D, SP_F32, kp, 1}, OutOperand{p.D, SP_F32, kp}, false,
                    status_dev, s, &sd, 2.0 * (double)Tc * d * k));
    } else if (decay_z) {
      // h of this chunk sits in the state, transposed ([k, Tc], tokens contiguous): written by the last step's update,
      // or gathered now
      __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(st->H_next) + (size_t)t0 * ldh_next;
      {
        SkipScope unless_stale(h_ready);
        CU(launch_gather_ht(Zc, Tc, n, k, p.grp_base, p.grp_mask, Hc, Tc, s));
      }
      MatRef hn{Hc, cdt, Tc};
      SPCHK(contract(Tc, d, k, -1.0, hn, false, w2, true, 1.0, yc, e, false, acc64, bf16, status_dev, s));
    } else {
      CU(launch_prep_h(Zc, Uc, Gc, p.H, cdt, Tc, n, kp, k, idx, s));
      SPCHK(contract(Tc, d, k, -1.0, h, true, w2, true, 1.0, yc, e, false, acc64, bf16, status_dev, s));
    }
    if (!split_h) SPCHK(contract(Tc, k, d, 1.0, e, true, qt, true, 0.0, dd, dd, false, acc64, bf16, status_dev, s));
    if (z1_ahead) {}   // already there for all tokens
    else if (bf16) SPCHK(contract_split_weights(Tc, k, d, xc, p.W1b, w1, z1, status_dev, s));
    else SPCHK(contract(Tc, k, d, 1.0, xc, true, w1, true, 0.0, z1, z1, false, acc64, false, status_dev, s));
    UpdateArgs ua;
    ua.Z = Zc; ua.U = Uc; ua.gate = Gc; ua.z1 = z1_ahead ? p.z1_all + (size_t)t0 * kp : p.z1; ua.D = p.D; ua.ldk = kp; ua.k = k; ua.grp_base = p.grp_base;
    ua.grp_mask = p.grp_mask; ua.A_out = p.Ac; ua.Zb_out = bf16 ? p.Zb : nullptr;
    ua.out_dtype = cdt; ua.T = Tc; ua.n = n; ua.alpha = (float)prm->alpha; ua.beta = (float)prm->beta;
    ua.z_rule = prm->z_rule; ua.partial = p.partial; ua.absA_part = p.absA_part;
    // bf16 storage: the update writes A transposed (channels x tokens), which makes the token dimension the
    // contiguous one of both operands of A A^T and of the A operand of Ypre A^T; the row-major A is only needed
    // when the objective is reported.  The row pitch is a multiple of 16 bytes.
    const int64_t Tld = (Tc + 7) / 8 * 8;
    const bool a_transposed = bf16 && n % 4 == 0 && !(rep_dev && prm->compute_objective) && Tld <= p.chunk;
    if (a_transposed) { ua.At_out = p.Ac; ua.ldt = Tld; }
    if (decay) ua.at_kept_first = 1;     // (the pruned rows are still needed: G_A[pruned, kept] is contracted anew)
    if (decay_z) {
      // the copy of Z for R1 and the next step's h are written transposed, by the same kernel
      ua.Zb_out = nullptr;
      ua.Zt_out = p.Zb;
      ua.Ht_out = reinterpret_cast<__nv_bfloat16*>(st->H_next) + (size_t)t0 * ldh_next;
      ua.zt_pruned_flag = h_ready + 1;       // the pruned rows of R1 are contracted only in a step that found h stale
    }
    const int nblk = decay_z ? fused_update_next_grid(Tc, n, &ua.row_blocks) : fused_update_grid(Tc, n, &ua.row_blocks);
    CU(launch_fused_update(ua, s));
    if (rep_dev) CU(reduce_report(p.partial, nblk, rep_dev, ci > 0, prm->alpha, s));
    if (rep_dev && prm->compute_objective) {
      // alpha |Ypre - W2 A|^2 of the new A: one more product per chunk, only on request
      MatRef w2f = bf16 ? MatRef{p.W2fb, SP_BF16, n} : MatRef{st->W2, SP_F32, n};
      MatRef eo{p.Eo, SP_F32, d};
      SPCHK(contract(Tc, d, n, -1.0, ac, true, w2f, true, 1.0, yc, eo, false, acc64, bf16, status_dev, s));
      CU(sumsq_accumulate(p.Eo, d, Tc, d, prm->alpha, &rep_dev->res_out, ci > 0, p.partial + (size_t)p.nblocks * 4, s));
    }
    CU(reduce_col_partials(p.absA_part, decay_z ? fused_update_next_partial_rows(ua.row_blocks) : ua.row_blocks, n,
                           st->absA, ci > 0, s));
    // accumulators of the new auxiliary variables
    if (decay) {
      // rows of A^T in "kept first" order: [0, k) kept, [k, n) pruned
      MatRef act{p.Ac, cdt, Tld};
      MatRef actp{reinterpret_cast<const __nv_bfloat16*>(p.Ac) + (size_t)k * Tld, cdt, Tld};
      MatRef gp{st->G_A_perm, SP_F32, n}, gpp{st->G_A_perm + (size_t)k * n + k, SP_F32, n};
      MatRef r2k{st->R2_perm, SP_F32, n}, r2p{st->R2_perm + k, SP_F32, n};
      SPCHK(contract(n, k, Tc, 1.0, act, true, act, true, acc, gp, gp, true, acc64, bf16, status_dev, s));
      SPCHK(contract(d, k, Tc, 1.0, yc, false, act, true, acc, r2k, r2k, false, acc64, bf16, status_dev, s));
      {
        SkipScope unless_changed(order_same);
        SPCHK(contract(n - k, n - k, Tc, 1.0, actp, true, actp, true, acc, gpp, gpp, true, acc64, bf16, status_dev, s));
        SPCHK(contract(d, n - k, Tc, 1.0, yc, false, actp, true, acc, r2p, r2p, false, acc64, bf16, status_dev, s));
      }
    } else if (a_transposed) {
      MatRef act{p.Ac, cdt, Tld};
      SPCHK(contract(n, n, Tc, 1.0, act, true, act, true, acc, ga, ga, true, acc64, bf16, status_dev, s));
      SPCHK(contract(d, n, Tc, 1.0, yc, false, act, true, acc, r2, r2, false, acc64, bf16, status_dev, s));
    } else {
      SPCHK(contract(n, n, Tc, 1.0, ac, false, ac, false, acc, ga, ga, true, acc64, bf16, status_dev, s));
      SPCHK(contract(d, n, Tc, 1.0, yc, false, ac, false, acc, r2, r2, false, acc64, bf16, status_dev, s));
    }
    if (decay_z) {
      MatRef zt{p.Zb, cdt, Tld}, ztp{reinterpret_cast<const __nv_bfloat16*>(p.Zb) + (size_t)k * Tld, cdt, Tld};
      MatRef r1k{st->R1_perm, SP_F32, d}, r1p{st->R1_perm + (size_t)k * d, SP_F32, d};
      SPCHK(contract(k, d, Tc, 1.0, zt, true, xc, false, acc, r1k, r1k, false, acc64, bf16, status_dev, s));
      {
        SkipScope unless_stale(h_ready);
        SPCHK(contract(n - k, d, Tc, 1.0, ztp, true, xc, false, acc, r1p, r1p, false, acc64, bf16, status_dev, s));
      }
    } else {
      SPCHK(contract(n, d, Tc, 1.0, zb, false, xc, false, acc, r1, r1, false, acc64, bf16, status_dev, s));
    }
  }
  if (decay) {
    // the accumulators in channel order for the next step's weight phase and for the caller
    CU(unpermute_gram(st->G_A_perm, st->decay_tag + 8, n, st->G_A, s));
    CU(unpermute_cols(st->R2_perm, st->decay_tag + 8, d, n, st->R2, s));
    if (decay_z) CU(unpermute_rows(st->R1_perm, st->decay_tag + 8, n, d, st->R1, s));
  } else {
    CU(symmetrize_lower(st->G_A, n, n, s));
  }
  join_guard.armed = false;
  return SP_OK;
}

sp_status sp_admm_step(const sp_ffn_module* m, sp_ffn_state* st, const sp_admm_params* prm, sp_step_report* rep_dev,
                       int32_t* status_dev, void* ws, size_t ws_bytes, void* stream) {
  return admm_step_impl(m, st, prm, rep_dev, status_dev, ws, ws_bytes, stream, false);
}

sp_status sp_admm_scores(const sp_ffn_module* m, sp_ffn_state* st, const sp_admm_params* prm, int32_t* status_dev,
                         void* ws, size_t ws_bytes, void* stream) {
  return admm_step_impl(m, st, prm, nullptr, status_dev, ws, ws_bytes, stream, true);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------ attention module
namespace {

// A token-major tensor seen as one [T, d_h] slice per (head, sequence) pair, or a [pairs, T, T] tensor; `planes`
// whole copies `plane` elements apart (bf16 hi / lo parts).
struct BMat {
  const void* ptr;
  int32_t dt;
  int64_t ld, s0, s1;   // leading dimension; element stride of the head (b0) and sequence (b1) index
  int planes = 1;
  int64_t plane = 0;
};

// C_b = alpha * sum over segments A_b[plane pa] B_b[plane pb] + beta * Cin_b for all nb0 x nb1 pairs.
// bf16 operands: one batched tensor-core launch.  fp32 operands (fp32 mode): plane 0 holds the full value, the
// segments collapse to one product per pair on the CUDA cores with fp64 accumulation.
sp_status bcontract(int64_t M, int64_t N, int64_t K, double alpha, BMat A, bool a_kmajor, BMat B, bool b_kmajor,
                    int nseg, const int* pa, const int* pb, double beta, BMat Cin, BMat C, int64_t c_lo_off, int nb0,
                    int nb1, int32_t* status, cudaStream_t s) {
  if (M <= 0 || N <= 0 || nb0 <= 0 || nb1 <= 0) return SP_OK;
  if (A.dt == SP_BF16 && B.dt == SP_BF16) {
    TcOperand ta{A.ptr, A.ld, a_kmajor}, tb{B.ptr, B.ld, b_kmajor};
    TcSegments sg;
    sg.nseg = nseg;
    for (int i = 0; i < nseg; ++i) { sg.a_p[i] = pa[i]; sg.b_p[i] = pb[i]; }
    TcBatch bt;
    bt.nb0 = nb0; bt.nb1 = nb1;
    bt.a_s0 = A.s0; bt.a_s1 = A.s1; bt.b_s0 = B.s0; bt.b_s1 = B.s1;
    bt.c_s0 = C.s0; bt.c_s1 = C.s1; bt.cin_s0 = Cin.s0; bt.cin_s1 = Cin.s1;
    bt.a_planes = A.planes; bt.a_plane = A.plane; bt.b_planes = B.planes; bt.b_plane = B.plane;
    OutOperand out{const_cast<void*>(C.ptr), C.dt, C.ld};
    out.lo_off = c_lo_off;
    return gemm_tc(M, N, K, (float)alpha, ta, tb, (float)beta, Operand{Cin.ptr, Cin.dt, Cin.ld, 1}, out, false, status,
                   s, &sg, 2.0 * (double)M * N * K * nb0 * nb1, 0, &bt);
  }
  for (int b1 = 0; b1 < nb1; ++b1)
    for (int b0 = 0; b0 < nb0; ++b0) {
      auto at = [&](const BMat& m) {
        return reinterpret_cast<const uint8_t*>(m.ptr) + ((size_t)b0 * m.s0 + (size_t)b1 * m.s1) * dtype_size(m.dt);
      };
      Operand a{at(A), A.dt, a_kmajor ? A.ld : 1, a_kmajor ? 1 : A.ld};
      Operand b{at(B), B.dt, b_kmajor ? 1 : B.ld, b_kmajor ? B.ld : 1};
      Operand cin{Cin.ptr ? at(Cin) : nullptr, Cin.dt, Cin.ld, 1};
      OutOperand out{const_cast<uint8_t*>(at(C)), C.dt, C.ld};
      CU(gemm_simt(M, N, K, alpha, a, b, beta, cin, out, false, true, s));
    }
  return SP_OK;
}

struct MhaPlan {
  int64_t d, H, T, dh, sc, cap;   // cap = tokens of a full chunk
  bool bf16;
  SolveBufs sb;
  float *Cf, *RW, *MC;            // W_O^T W_O; [W_O; I] right-hand sides; [M1; Cinv] = [W_O; I] (W_O^T W_O + I)^-1
  void *Wqs, *Wks, *Wvs, *Wos, *M1s, *Cis;   // bf16 hi | lo forms of the weights ([d, 2 pad64(d)])
  float *Tq, *Tk, *Vf, *Gq, *Gk;  // [cap, d] fp32
  void *Vs, *Zqs, *Zks;           // bf16 hi / lo planes [2][cap, d]
  void *Rb, *Hd;                  // R = A_attn - P V ([cap, d]); head outputs as hi | lo ([cap, 2 pad64(d)])
  float *S, *G;                   // [sc H, T, T] fp32
  void* Pb;                       // [2][sc H, T, T] bf16: hi / lo planes of P; plane 0 later holds dS
  double* sums;
  float *eta_a, *eta_z;
  size_t bytes;
};

MhaPlan plan_mha(void* ws, int64_t d, int64_t H, int64_t T, int64_t n_seq, int64_t seq_chunk, int32_t cdt) {
  MhaPlan p;
  p.d = d; p.H = H; p.T = T; p.dh = H > 0 ? d / H : d;
  p.sc = seq_chunk > 0 ? seq_chunk : 1;
  if (p.sc > n_seq) p.sc = n_seq;
  if (p.sc < 1) p.sc = 1;
  p.cap = p.sc * T;
  p.bf16 = cdt == SP_BF16;
  const size_t tsize = p.bf16 ? 4 : 8;
  const size_t dp = (size_t)split_kpad(d);
  Carver c(ws);
  p.sb = carve_solve(c, d, 2 * d, tsize);
  p.Cf = c.take<float>((size_t)d * d);
  p.RW = c.take<float>((size_t)2 * d * d);
  p.MC = c.take<float>((size_t)2 * d * d);
  p.Wqs = p.Wks = p.Wvs = p.Wos = p.M1s = p.Cis = nullptr;
  if (p.bf16) {
    p.Wqs = c.take_bytes((size_t)d * 2 * dp * 2); p.Wks = c.take_bytes((size_t)d * 2 * dp * 2);
    p.Wvs = c.take_bytes((size_t)d * 2 * dp * 2); p.Wos = c.take_bytes((size_t)d * 2 * dp * 2);
    p.M1s = c.take_bytes((size_t)d * 2 * dp * 2); p.Cis = c.take_bytes((size_t)d * 2 * dp * 2);
  }
  const size_t tok = (size_t)p.cap * d, tt = (size_t)p.sc * H * T * T;
  p.Tq = c.take<float>(tok); p.Tk = c.take<float>(tok); p.Vf = c.take<float>(tok);
  p.Gq = c.take<float>(tok); p.Gk = c.take<float>(tok);
  p.Vs = p.Zqs = p.Zks = p.Pb = nullptr;
  if (p.bf16) {
    p.Vs = c.take_bytes(2 * tok * 2); p.Zqs = c.take_bytes(2 * tok * 2); p.Zks = c.take_bytes(2 * tok * 2);
    p.Pb = c.take_bytes(2 * tt * 2);      // hi / lo planes
  }
  p.Rb = c.take_bytes(tok * (p.bf16 ? 2 : 4));
  p.Hd = c.take_bytes((size_t)p.cap * (p.bf16 ? 2 * dp * 2 : (size_t)d * 4));
  p.S = c.take<float>(tt);
  p.G = c.take<float>(tt);
  p.sums = c.take<double>((size_t)p.sc * H);
  p.eta_a = c.take<float>((size_t)p.sc * H);
  p.eta_z = c.take<float>((size_t)p.sc * H);
  p.bytes = align_up(c.off, 256);
  return p;
}

sp_status check_mha(const sp_mha_module* m, const sp_mha_state* st) {
  if (!m || !st) return SP_ERR_INVALID_ARG;
  if (m->d < 1 || m->n_heads < 1 || m->T < 1 || m->n_seq < 1 || m->d % m->n_heads != 0) return SP_ERR_SHAPE;
  const int64_t N = m->n_seq * m->T;
  if (!m->X.ptr || !m->Ypre.ptr) return SP_ERR_INVALID_ARG;
  if (!valid_act_dtype(m->X.dtype) || m->Ypre.dtype != m->X.dtype) return SP_ERR_DTYPE;
  if (m->X.rows != N || m->X.cols != m->d || m->X.ld != m->d) return SP_ERR_SHAPE;
  if (m->Ypre.rows != N || m->Ypre.cols != m->d || m->Ypre.ld != m->d) return SP_ERR_SHAPE;
  const sp_mat* w[4] = {&m->Wq, &m->Wk, &m->Wv, &m->Wo};
  for (const sp_mat* x : w) {
    if (!x->ptr) return SP_ERR_INVALID_ARG;
    if (x->dtype != SP_F32) return SP_ERR_DTYPE;
    if (x->rows != m->d || x->cols != m->d || x->ld != m->d) return SP_ERR_SHAPE;
  }
  if (!st->Zq || !st->Zk || !st->P || !st->Aattn) return SP_ERR_INVALID_ARG;
  {
    const int have = (st->G_X != nullptr) + (st->R_Q != nullptr) + (st->R_K != nullptr) + (st->G_attn != nullptr) +
                     (st->R_O != nullptr);
    if (have != 0 && have != 5) return SP_ERR_INVALID_ARG;
  }
  // the tensor-core path slices heads out of token-major tensors with 16-byte aligned strides
  if (m->X.dtype == SP_BF16 && ((m->d / m->n_heads) % 8 != 0 || m->T % 8 != 0)) return SP_ERR_ALIGNMENT;
  if (misaligned(st->Zq, 16) || misaligned(st->Zk, 16) || misaligned(st->P, 16) || misaligned(st->Aattn, 16) ||
      misaligned(m->X.ptr, 16) || misaligned(m->Ypre.ptr, 16))
    return SP_ERR_ALIGNMENT;
  return SP_OK;
}

// X W^T for all tokens of a chunk with fp32 weights W [d, d] (bf16 mode: hi | lo split Ws), fp32 result [Tc, d].
sp_status project(const MhaPlan& p, MatRef xc, const void* Ws, const sp_mat& W, float* out, int64_t Tc, int32_t* status,
                  cudaStream_t s) {
  MatRef o{out, SP_F32, p.d};
  if (p.bf16) return contract_split_weights(Tc, p.d, p.d, xc, Ws, MatRef{W.ptr, SP_F32, W.ld}, o, status, s);
  return contract(Tc, p.d, p.d, 1.0, xc, true, MatRef{W.ptr, SP_F32, W.ld}, true, 0.0, o, o, false, true, false, status, s);
}

// The accumulators of the weight recoveries over one chunk of tokens (first chunk: overwrite).  bf16 mode: Zq, Zk and
// Aattn enter as their bf16 roundings (the precision model of the FFN path's accumulators): the hi planes of Zq / Zk
// kept for the logits, a bf16 copy of Aattn in the buffer of R.
sp_status mha_accumulate(const MhaPlan& p, const sp_mha_module* m, sp_mha_state* st, MatRef xc, MatRef yc, const float* Zq,
                         const float* Zk, const float* Aat, int64_t Tc, bool first, int32_t* status, cudaStream_t s) {
  if (!st->G_X) return SP_OK;
  (void)m;
  const int64_t d = p.d;
  const double acc = first ? 0.0 : 1.0;
  const bool bf16 = p.bf16, acc64 = !bf16;
  MatRef zq{Zq, SP_F32, d}, zk{Zk, SP_F32, d}, aa{Aat, SP_F32, d};
  if (bf16) {
    // the hi planes of Zq / Zk are current (written by the last update, or by the split at the start of the chunk)
    CU(split_planes(Aat, Tc * d, p.Rb, 0, s));
    zq = MatRef{p.Zqs, SP_BF16, d};
    zk = MatRef{p.Zks, SP_BF16, d};
    aa = MatRef{p.Rb, SP_BF16, d};
  }
  MatRef gx{st->G_X, SP_F32, d}, rq{st->R_Q, SP_F32, d}, rk{st->R_K, SP_F32, d}, ga{st->G_attn, SP_F32, d},
      ro{st->R_O, SP_F32, d};
  SPCHK(contract(d, d, Tc, 1.0, xc, false, xc, false, acc, gx, gx, true, acc64, bf16, status, s));
  SPCHK(contract(d, d, Tc, 1.0, zq, false, xc, false, acc, rq, rq, false, acc64, bf16, status, s));
  SPCHK(contract(d, d, Tc, 1.0, zk, false, xc, false, acc, rk, rk, false, acc64, bf16, status, s));
  SPCHK(contract(d, d, Tc, 1.0, aa, false, aa, false, acc, ga, ga, true, acc64, bf16, status, s));
  SPCHK(contract(d, d, Tc, 1.0, yc, false, aa, false, acc, ro, ro, false, acc64, bf16, status, s));
  return SP_OK;
}

constexpr int kSegHH[1] = {0};
constexpr int kSeg3A[3] = {0, 1, 0}, kSeg3B[3] = {0, 0, 1};   // hi.hi, lo.hi, hi.lo

}  // namespace

extern "C" {

size_t sp_mha_workspace_bytes(int64_t d, int64_t n_heads, int64_t T, int64_t n_seq, int64_t seq_chunk, int32_t dtype) {
  if (d < 1 || n_heads < 1 || T < 1 || n_seq < 1) return 0;
  return plan_mha(nullptr, d, n_heads, T, n_seq, seq_chunk, dtype).bytes + 256;
}

// Shared body of sp_mha_init (init = true: the forward definition) and sp_mha_step.
static sp_status mha_impl(const sp_mha_module* m, sp_mha_state* st, const sp_mha_params* prm, bool init,
                          int64_t seq_chunk, int32_t* status_dev, void* ws, size_t ws_bytes, void* stream) {
  SPCHK(check_mha(m, st));
  const int64_t d = m->d, H = m->n_heads, T = m->T, n_seq = m->n_seq, dh = d / H;
  const int32_t cdt = m->X.dtype;
  if (!prm) return SP_ERR_INVALID_ARG;
  if (!init) {
    if (!(prm->alpha > 0.0) || !(prm->beta > 0.0) || prm->a_steps < 0 || prm->z_steps < 0 || !(prm->eta_z > 0.0) ||
        prm->eta_z > 1.0 || prm->seq_chunk < 0)
      return SP_ERR_INVALID_ARG;
    seq_chunk = prm->seq_chunk;
  }
  if (seq_chunk < 0) return SP_ERR_INVALID_ARG;
  if (!ws || ws_bytes < plan_mha(nullptr, d, H, T, n_seq, seq_chunk, cdt).bytes) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  MhaPlan p = plan_mha(ws, d, H, T, n_seq, seq_chunk, cdt);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const bool bf16 = p.bf16, causal = prm->causal != 0;
  const int64_t dp = split_kpad(d);
  const size_t esz = bf16 ? 2 : 4;
  const double inv_sqrt = 1.0 / sqrt((double)dh);
  const int64_t TT = T * T;
  const int32_t odt = bf16 ? SP_BF16 : SP_F32;      // type of the operand copies
  const int64_t plane = p.cap * d;                   // distance of the lo plane of [cap, d] operand copies

  // ---- operands that do not depend on the tokens
  if (bf16) {
    CU(split_bf16(reinterpret_cast<const float*>(m->Wq.ptr), d, nullptr, d, d, dp, p.Wqs, s));
    CU(split_bf16(reinterpret_cast<const float*>(m->Wk.ptr), d, nullptr, d, d, dp, p.Wks, s));
    CU(split_bf16(reinterpret_cast<const float*>(m->Wv.ptr), d, nullptr, d, d, dp, p.Wvs, s));
    if (init) CU(split_bf16(reinterpret_cast<const float*>(m->Wo.ptr), d, nullptr, d, d, dp, p.Wos, s));
  }
  if (!init) {
    // Eq. (86): a_attn = (W_O^T W_O + I)^-1 (W_O^T ypre + heads); token-major: A_attn = Ypre M1 + Hd Cinv with
    // [M1; Cinv] = [W_O; I] (W_O^T W_O + I)^-1, one regularised solve with 2 d right-hand sides
    MatRef wo{m->Wo.ptr, SP_F32, d}, cf{p.Cf, SP_F32, d};
    SPCHK(contract(d, d, d, 1.0, wo, false, wo, false, 0.0, cf, cf, true, true, false, status_dev, s));
    CU(symmetrize_lower(p.Cf, d, d, s));
    CU(cudaMemcpyAsync(p.RW, m->Wo.ptr, (size_t)d * d * sizeof(float), cudaMemcpyDeviceToDevice, s));
    CU(set_identity(p.RW + (size_t)d * d, d, d, s));
    CU(effective_ridge(nullptr, 0, 1, 1.0, 0, p.sb.rho, s));
    if (bf16) SPCHK(ridge_core<float>(p.RW, d, p.Cf, d, 2 * d, d, nullptr, d, p.sb.rho, p.MC, d, p.sb, status_dev, s));
    else SPCHK(ridge_core<double>(p.RW, d, p.Cf, d, 2 * d, d, nullptr, d, p.sb.rho, p.MC, d, p.sb, status_dev, s));
    if (bf16) {
      CU(split_bf16(p.MC, d, nullptr, d, d, dp, p.M1s, s));
      CU(split_bf16(p.MC + (size_t)d * d, d, nullptr, d, d, dp, p.Cis, s));
    }
  }

  for (int64_t q0 = 0; q0 < n_seq; q0 += p.sc) {
    const int64_t nq = (n_seq - q0 < p.sc) ? n_seq - q0 : p.sc;
    const int64_t t0 = q0 * T, Tc = nq * T;
    const int nb0 = (int)H, nb1 = (int)nq;
    const int64_t pairs = nq * H;
    MatRef xc{reinterpret_cast<const uint8_t*>(m->X.ptr) + (size_t)t0 * d * esz, cdt, d};
    MatRef yc{reinterpret_cast<uint8_t*>(m->Ypre.ptr) + (size_t)t0 * d * esz, cdt, d};
    float* Zq = st->Zq + (size_t)t0 * d;
    float* Zk = st->Zk + (size_t)t0 * d;
    float* Aat = st->Aattn + (size_t)t0 * d;
    float* P = st->P + (size_t)q0 * H * TT;
    // views: [T, d_h] slices of token-major tensors, and [pairs, T, T] tensors
    auto tokv = [&](const void* ptr, int32_t dt, int64_t ld, int planes, int64_t pl) {
      return BMat{ptr, dt, ld, dh, T * ld, planes, pl};
    };
    auto ttv = [&](const void* ptr, int32_t dt) { return BMat{ptr, dt, T, TT, H * TT, 1, 0}; };
    const int64_t pplane = p.sc * H * TT;            // distance of the lo plane of the bf16 copy of P
    const BMat Pop = bf16 ? BMat{p.Pb, SP_BF16, T, TT, H * TT, 2, pplane} : ttv(P, SP_F32);
    const BMat none{nullptr, SP_F32, 0, 0, 0, 1, 0};

    // targets of the projections (and, at initialisation, the projections themselves)
    SPCHK(project(p, xc, p.Wqs, m->Wq, init ? Zq : p.Tq, Tc, status_dev, s));
    SPCHK(project(p, xc, p.Wks, m->Wk, init ? Zk : p.Tk, Tc, status_dev, s));
    SPCHK(project(p, xc, p.Wvs, m->Wv, p.Vf, Tc, status_dev, s));
    const void* Vop = p.Vf;
    const void* Zqop = Zq;
    const void* Zkop = Zk;
    if (bf16) {
      CU(split_planes(p.Vf, Tc * d, p.Vs, plane, s));
      CU(split_planes(Zq, Tc * d, p.Zqs, plane, s));
      CU(split_planes(Zk, Tc * d, p.Zks, plane, s));
      Vop = p.Vs; Zqop = p.Zqs; Zkop = p.Zks;
    }
    const int np2 = bf16 ? 2 : 1;
    const BMat Vv = tokv(Vop, odt, d, np2, plane), Zqv = tokv(Zqop, odt, d, np2, plane), Zkv = tokv(Zkop, odt, d, np2, plane);

    // logits S = Zq_i Zk_i^T / sqrt(d_h) and Phi = softmax(S)
    SPCHK(bcontract(T, T, dh, inv_sqrt, Zqv, true, Zkv, true, bf16 ? 3 : 1, kSeg3A, kSeg3B, 0.0, none, ttv(p.S, SP_F32), 0,
                    nb0, nb1, status_dev, s));
    if (init) {
      // forward definition: P = softmax(S), heads = P V, Ypre = heads W_O^T
      CU(mha_softmax_rows(p.S, pairs, (int)T, causal, p.Pb, pplane, s));
      CU(cudaMemcpyAsync(P, p.S, (size_t)pairs * TT * sizeof(float), cudaMemcpyDeviceToDevice, s));
      SPCHK(bcontract(T, dh, T, 1.0, Pop, true, Vv, false, bf16 ? 3 : 1, kSeg3A, kSeg3B, 0.0, none,
                      tokv(Aat, SP_F32, d, 1, 0), 0, nb0, nb1, status_dev, s));
      if (bf16) {
        CU(split_bf16(Aat, d, nullptr, Tc, d, dp, p.Hd, s));
        TcOperand ta{p.Hd, 2 * dp, true}, tb{p.Wos, 2 * dp, true};
        ta.kext = tb.kext = 2 * dp;
        TcSegments sg;
        sg.nseg = 3;
        sg.a_k[1] = (int32_t)dp;
        sg.b_k[2] = (int32_t)dp;
        SPCHK(gemm_tc(Tc, d, d, 1.f, ta, tb, 0.f, Operand{yc.ptr, cdt, d, 1}, OutOperand{const_cast<void*>(yc.ptr), cdt, d},
                      false, status_dev, s, &sg, 2.0 * (double)Tc * d * d));
      } else {
        MatRef a{Aat, SP_F32, d};
        SPCHK(contract(Tc, d, d, 1.0, a, true, MatRef{m->Wo.ptr, SP_F32, d}, true, 0.0, yc, yc, false, true, false,
                       status_dev, s));
      }
      SPCHK(mha_accumulate(p, m, st, xc, yc, Zq, Zk, Aat, Tc, q0 == 0, status_dev, s));
      continue;
    }

    // ---- Eq. (85): gradient steps on P with Phi fixed
    CU(mha_softmax_rows(p.S, pairs, (int)T, causal, nullptr, 0, s));
    CU(mha_step_sizes(p.Vf, nullptr, d, nq, (int)T, (int)dh, (int)H, 0, prm->alpha, prm->beta, 0.0, p.sums, p.eta_a, s));
    if (bf16) CU(split_planes(P, pairs * TT, p.Pb, pplane, s));
    const BMat Rv = tokv(p.Rb, odt, d, 1, 0);
    for (int it = 0; it < prm->a_steps; ++it) {
      // R = A_attn_i - P V_i ; G1 = R V_i^T
      SPCHK(bcontract(T, dh, T, -1.0, Pop, true, Vv, false, bf16 ? 3 : 1, kSeg3A, kSeg3B, 1.0, tokv(Aat, SP_F32, d, 1, 0),
                      Rv, 0, nb0, nb1, status_dev, s));
      SPCHK(bcontract(T, T, dh, 1.0, Rv, true, Vv, true, 1, kSegHH, kSegHH, 0.0, none, ttv(p.G, SP_F32), 0, nb0, nb1,
                      status_dev, s));
      CU(mha_p_update(P, p.S, p.G, p.eta_a, pairs, (int)T, prm->alpha, prm->beta, p.Pb, pplane, s));
    }
    // ---- Eq. (86): head outputs Hd = P V, then A_attn = Ypre M1 + Hd Cinv
    {
      BMat hv = bf16 ? tokv(p.Hd, SP_BF16, 2 * dp, 1, 0) : tokv(p.Hd, SP_F32, d, 1, 0);
      SPCHK(bcontract(T, dh, T, 1.0, Pop, true, Vv, false, bf16 ? 3 : 1, kSeg3A, kSeg3B, 0.0, none, hv, bf16 ? dp : 0,
                      nb0, nb1, status_dev, s));
      if (bf16) {
        TcOperand ya{yc.ptr, d, true}, mb{p.M1s, 2 * dp, false};
        mb.kext = d;
        mb.mnext = 2 * dp;
        TcSegments s1;
        s1.nseg = 2;
        s1.b_mn[1] = (int32_t)dp;
        SPCHK(gemm_tc(Tc, d, d, 1.f, ya, mb, 0.f, Operand{Aat, SP_F32, d, 1}, OutOperand{Aat, SP_F32, d}, false,
                      status_dev, s, &s1, 2.0 * (double)Tc * d * d));
        TcOperand ha{p.Hd, 2 * dp, true}, cb{p.Cis, 2 * dp, false};
        ha.kext = 2 * dp;
        cb.kext = d;
        cb.mnext = 2 * dp;
        TcSegments s2;
        s2.nseg = 3;
        s2.a_k[1] = (int32_t)dp;
        s2.b_mn[2] = (int32_t)dp;
        SPCHK(gemm_tc(Tc, d, d, 1.f, ha, cb, 1.f, Operand{Aat, SP_F32, d, 1}, OutOperand{Aat, SP_F32, d}, false,
                      status_dev, s, &s2, 2.0 * (double)Tc * d * d));
      } else {
        MatRef a{Aat, SP_F32, d}, m1{p.MC, SP_F32, d}, ci{p.MC + (size_t)d * d, SP_F32, d}, hd{p.Hd, SP_F32, d};
        SPCHK(contract(Tc, d, d, 1.0, yc, true, m1, false, 0.0, a, a, false, true, false, status_dev, s));
        SPCHK(contract(Tc, d, d, 1.0, hd, true, ci, false, 1.0, a, a, false, true, false, status_dev, s));
      }
    }
    // ---- Eq. (87): joint gradient steps on (Zq, Zk) through the softmax
    for (int it = 0; it < prm->z_steps; ++it) {
      SPCHK(bcontract(T, T, dh, inv_sqrt, Zqv, true, Zkv, true, bf16 ? 3 : 1, kSeg3A, kSeg3B, 0.0, none,
                      ttv(p.G, SP_F32), 0, nb0, nb1, status_dev, s));
      CU(mha_softmax_backward_rows(p.G, P, pairs, (int)T, causal, prm->beta, p.Pb, s));
      const BMat dS = bf16 ? ttv(p.Pb, SP_BF16) : ttv(p.G, SP_F32);
      // gq = dS Zk_i / sqrt(d_h), gk = dS^T Zq_i / sqrt(d_h) (hi parts of the operands)
      BMat Zk1 = Zkv, Zq1 = Zqv;
      Zk1.planes = Zq1.planes = 1;
      SPCHK(bcontract(T, dh, T, inv_sqrt, dS, true, Zk1, false, 1, kSegHH, kSegHH, 0.0, none, tokv(p.Gq, SP_F32, d, 1, 0),
                      0, nb0, nb1, status_dev, s));
      SPCHK(bcontract(T, dh, T, inv_sqrt, dS, false, Zq1, false, 1, kSegHH, kSegHH, 0.0, none, tokv(p.Gk, SP_F32, d, 1, 0),
                      0, nb0, nb1, status_dev, s));
      CU(mha_step_sizes(Zq, Zk, d, nq, (int)T, (int)dh, (int)H, 1, prm->alpha, prm->beta, prm->eta_z, p.sums, p.eta_z, s));
      CU(mha_z_update(Zq, Zk, p.Gq, p.Gk, p.Tq, p.Tk, p.eta_z, Tc, (int)d, (int)T, (int)dh, prm->alpha,
                      bf16 ? p.Zqs : nullptr, bf16 ? p.Zks : nullptr, plane, s));
    }
    SPCHK(mha_accumulate(p, m, st, xc, yc, Zq, Zk, Aat, Tc, q0 == 0, status_dev, s));
  }
  if (st->G_X) {
    CU(symmetrize_lower(st->G_X, d, d, s));
    CU(symmetrize_lower(st->G_attn, d, d, s));
  }
  return SP_OK;
}

sp_status sp_mha_init(const sp_mha_module* m, sp_mha_state* st, int32_t causal, int64_t seq_chunk, int32_t* status_dev,
                      void* ws, size_t ws_bytes, void* stream) {
  sp_mha_params prm;
  memset(&prm, 0, sizeof(prm));
  prm.causal = causal;
  return mha_impl(m, st, &prm, true, seq_chunk, status_dev, ws, ws_bytes, stream);
}

sp_status sp_mha_step(const sp_mha_module* m, sp_mha_state* st, const sp_mha_params* p, int32_t* status_dev, void* ws,
                      size_t ws_bytes, void* stream) {
  return mha_impl(m, st, p, false, 0, status_dev, ws, ws_bytes, stream);
}

// ---- recovery of W_V from the auxiliary head outputs
namespace {
struct ValueRefitPlan {
  int64_t dh, sc, cap;
  bool bf16;
  SolveBufs sb, sb2;   // two sets: the systems of the heads are independent and are solved two at a time
  void* Pb;     // bf16 mode: hi / lo planes of P of one chunk, [2][sc H, T, T]
  void* Ab;     // bf16 mode: Aattn of one chunk as bf16 hi | lo parts, [cap, 2 pad64(d)]
  void* R;      // regressors of one head and chunk: bf16 hi | lo [cap, 2 pad64(d)], or fp32 [cap, d]
  float* G;     // [H][d, d]   sum over sequences of R^T R per head (lower triangle)
  float* Cv;    // [H][d_h, d] sum over sequences of Aattn_i^T R per head
  // the heads' systems solved together (bf16 mode, d a multiple of the solver's block): see potrf_potrs_tc_batched
  bool batched;
  float *Gs_all, *dinv_all;
  void *P_all, *Xs_all;
  double* rho_all;
  size_t bytes;
};

ValueRefitPlan plan_value_refit(void* ws, int64_t d, int64_t H, int64_t T, int64_t n_seq, int64_t seq_chunk,
                                int32_t cdt) {
  ValueRefitPlan p;
  p.dh = H > 0 ? d / H : d;
  p.sc = seq_chunk > 0 ? seq_chunk : 1;
  if (p.sc > n_seq) p.sc = n_seq;
  if (p.sc < 1) p.sc = 1;
  p.cap = p.sc * T;
  p.bf16 = cdt == SP_BF16;
  Carver c(ws);
  p.sb = carve_solve(c, d, p.dh, p.bf16 ? 4 : 8);
  p.sb2 = carve_solve(c, d, p.dh, p.bf16 ? 4 : 8);
  p.Pb = p.bf16 ? c.take_bytes((size_t)2 * p.sc * H * T * T * 2) : nullptr;
  p.Ab = p.bf16 ? c.take_bytes((size_t)p.cap * 2 * split_kpad(d) * 2) : nullptr;
  p.R = c.take_bytes(p.bf16 ? (size_t)p.cap * 2 * split_kpad(d) * 2 : (size_t)p.cap * d * 4);
  p.G = c.take<float>((size_t)H * d * d);
  p.Cv = c.take<float>((size_t)d * d);
  p.batched = p.bf16 && d % kCholTcNB == 0;
  p.Gs_all = p.dinv_all = nullptr;
  p.P_all = p.Xs_all = nullptr;
  p.rho_all = nullptr;
  if (p.batched) {
    p.rho_all = c.take<double>((size_t)H);
    p.Gs_all = c.take<float>((size_t)H * (d + p.dh) * d);
    p.dinv_all = c.take<float>((size_t)H * dinv_elems(d));
    p.P_all = c.take_bytes((size_t)H * (d + p.dh) * 3 * d * 2);
    p.Xs_all = c.take_bytes((size_t)H * 2 * p.dh * 3 * kCholTcNB * 2);
  }
  p.bytes = align_up(c.off, 256);
  return p;
}
}  // namespace

size_t sp_mha_value_refit_workspace_bytes(int64_t d, int64_t n_heads, int64_t T, int64_t n_seq, int64_t seq_chunk,
                                          int32_t dtype) {
  if (d < 1 || n_heads < 1 || T < 1 || n_seq < 1) return 0;
  return plan_value_refit(nullptr, d, n_heads, T, n_seq, seq_chunk, dtype).bytes + 256;
}

sp_status sp_mha_value_refit(const sp_mha_module* m, const sp_mha_state* st, const uint8_t* head_mask_host, double rho,
                             int32_t rho_relative, int64_t seq_chunk, float* Wv_out, int64_t ldw, int32_t* status_dev,
                             void* ws, size_t ws_bytes, void* stream) {
  SPCHK(check_mha(m, st));
  if (!Wv_out || !(rho >= 0.0) || seq_chunk < 0) return SP_ERR_INVALID_ARG;
  const int64_t d = m->d, H = m->n_heads, T = m->T, n_seq = m->n_seq, dh = d / H;
  if (ldw < d) return SP_ERR_SHAPE;
  const int32_t cdt = m->X.dtype;
  if (!ws || ws_bytes < plan_value_refit(nullptr, d, H, T, n_seq, seq_chunk, cdt).bytes) return SP_ERR_WORKSPACE;
  if (misaligned(ws, 256)) return SP_ERR_ALIGNMENT;
  ValueRefitPlan p = plan_value_refit(ws, d, H, T, n_seq, seq_chunk, cdt);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const bool bf16 = p.bf16;
  const size_t esz = bf16 ? 2 : 4;
  const int64_t TT = T * T, dp = split_kpad(d);
  auto kept = [&](int64_t i) { return head_mask_host == nullptr || head_mask_host[i] != 0; };
  CU(cudaMemset2DAsync(Wv_out, (size_t)ldw * sizeof(float), 0, (size_t)d * sizeof(float), (size_t)d, s));

  // ---- per head: G_i = sum_s R^T R and C_i = sum_s Aattn_i^T R with the regressors R = P_i X of every sequence
  // (token-major: row q of R is sum_k P_i[q, k] x_k)
  for (int64_t q0 = 0; q0 < n_seq; q0 += p.sc) {
    const int64_t nq = (n_seq - q0 < p.sc) ? n_seq - q0 : p.sc;
    const int64_t t0 = q0 * T, Tc = nq * T, pairs = nq * H;
    const double acc = q0 > 0 ? 1.0 : 0.0;
    const uint8_t* xptr = reinterpret_cast<const uint8_t*>(m->X.ptr) + (size_t)t0 * d * esz;
    const float* Aat = st->Aattn + (size_t)t0 * d;
    const float* P = st->P + (size_t)q0 * H * TT;
    const int64_t pplane = p.sc * H * TT;
    if (bf16) {
      CU(split_planes(P, pairs * TT, p.Pb, pplane, s));
      CU(split_bf16(Aat, d, nullptr, Tc, d, dp, p.Ab, s));
    }
    const BMat none{nullptr, SP_F32, 0, 0, 0, 1, 0};
    for (int64_t i = 0; i < H; ++i) {
      if (!kept(i)) continue;
      float* Gi = p.G + (size_t)i * d * d;
      float* Ci = p.Cv + (size_t)i * dh * d;
      // one launch for the nq sequences of the chunk (the batch index b0 is not used: one head at a time)
      const BMat Xb{xptr, cdt, d, d, T * d, 1, 0};
      if (bf16) {
        const BMat Pi{reinterpret_cast<const __nv_bfloat16*>(p.Pb) + (size_t)i * TT, SP_BF16, T, TT, H * TT, 2, pplane};
        const BMat Rb{p.R, SP_BF16, 2 * dp, 2 * dp, T * 2 * dp, 1, 0};
        static const int pa[2] = {0, 1}, pb[2] = {0, 0};     // (P hi + P lo) X
        SPCHK(bcontract(T, d, T, 1.0, Pi, true, Xb, false, 2, pa, pb, 0.0, none, Rb, dp, 1, (int)nq, status_dev, s));
        // G_i (+)= R^T R with R = R_hi + R_lo: hi.hi, lo.hi, hi.lo; the token axis is K, both operands MN-major
        TcOperand ra{p.R, 2 * dp, false}, rb{p.R, 2 * dp, false};
        ra.kext = rb.kext = Tc;
        ra.mnext = rb.mnext = 2 * dp;
        TcSegments sg;
        sg.nseg = 3;
        sg.a_mn[1] = (int32_t)dp;
        sg.b_mn[2] = (int32_t)dp;
        SPCHK(gemm_tc(d, d, Tc, 1.f, ra, rb, (float)acc, Operand{Gi, SP_F32, d, 1}, OutOperand{Gi, SP_F32, d}, true,
                      status_dev, s, &sg, (double)d * d * Tc));
        // C_i (+)= Aattn_i^T R: the head's d_h columns of Aattn (hi | lo) against R (hi | lo): hi.hi, lo.hi, hi.lo
        TcOperand aa{reinterpret_cast<const __nv_bfloat16*>(p.Ab) + i * dh, 2 * dp, false};
        aa.kext = Tc;
        aa.mnext = dp + dh;      // the lo part of the head's columns sits dp columns to the right
        TcSegments sc2;
        sc2.nseg = 3;
        sc2.a_mn[1] = (int32_t)dp;
        sc2.b_mn[2] = (int32_t)dp;
        SPCHK(gemm_tc(dh, d, Tc, 1.f, aa, rb, (float)acc, Operand{Ci, SP_F32, d, 1}, OutOperand{Ci, SP_F32, d}, false,
                      status_dev, s, &sc2, 2.0 * (double)dh * d * Tc));
      } else {
        const BMat Pi{P + (size_t)i * TT, SP_F32, T, TT, H * TT, 1, 0};
        const BMat Rb{p.R, SP_F32, d, d, T * d, 1, 0};
        SPCHK(bcontract(T, d, T, 1.0, Pi, true, Xb, false, 1, kSegHH, kSegHH, 0.0, none, Rb, 0, 1, (int)nq, status_dev,
                        s));
        MatRef r{p.R, SP_F32, d}, g{Gi, SP_F32, d}, c{Ci, SP_F32, d}, a{Aat + i * dh, SP_F32, d};
        SPCHK(contract(d, d, Tc, 1.0, r, false, r, false, acc, g, g, true, true, false, status_dev, s));
        SPCHK(contract(dh, d, Tc, 1.0, a, false, r, false, acc, c, c, false, true, false, status_dev, s));
      }
    }
  }
  // ---- W_V,i = C_i (G_i + rho_i I)^-1, one regularised solve per kept head.
  if (p.batched) {
    // all kept heads' systems together: every step of the factorisation and of the sweep is one launch over them
    const int64_t a_bs = (d + dh) * d, d_bs = (int64_t)dinv_elems(d);
    int nk = 0;
    for (int64_t i = 0; i < H; ++i) {
      if (!kept(i)) continue;
      float* Gs = p.Gs_all + (size_t)nk * a_bs;
      CU(effective_ridge(p.G + (size_t)i * d * d, d, d, rho, rho_relative, p.rho_all + nk, s));
      CU(load_spd<float>(p.G + (size_t)i * d * d, d, d, p.rho_all + nk, Gs, d, s));
      CU(gather_cols<float>(p.Cv + (size_t)i * dh * d, d, nullptr, dh, d, Gs + (size_t)d * d, d, s));
      ++nk;
    }
    if (nk > 0) {
      ProfScope prof(PK_SOLVE, (double)nk * ((double)d * d * d / 3.0 + 2.0 * (double)dh * d * d), 0.0, s);
      SPCHK(potrf_potrs_tc_batched(p.Gs_all, d, dh, nk, a_bs, p.dinv_all, d_bs, p.P_all, p.Xs_all, status_dev, s));
    }
    nk = 0;
    for (int64_t i = 0; i < H; ++i) {
      if (!kept(i)) continue;
      const float* Xi = p.Gs_all + (size_t)nk * a_bs + (size_t)d * d;
      CU(scatter_cols<float>(Xi, d, nullptr, dh, d, d, Wv_out + (size_t)i * dh * ldw, ldw, s));
      ++nk;
    }
    return SP_OK;
  }
  // Otherwise one system at a time.  A solve is a chain of short kernels that leaves most SMs idle, and the heads'
  // systems are independent: they alternate between the caller's stream and the library's side stream, each with its
  // own buffers and assisting stream.
  SideStream* side = side_stream();
  JoinOnExit join_guard{side, s};
  if (side) {
    CU(cudaEventRecord(side->fork, s));
    CU(cudaStreamWaitEvent(side->stream, side->fork, 0));
  }
  int64_t turn = 0;
  for (int64_t i = 0; i < H; ++i) {
    if (!kept(i)) continue;
    const float* Gi = p.G + (size_t)i * d * d;
    const float* Ci = p.Cv + (size_t)i * dh * d;
    float* Wi = Wv_out + (size_t)i * dh * ldw;
    const bool on_side = side != nullptr && (turn++ & 1) != 0;
    cudaStream_t sq = on_side ? side->stream : s;
    SolveBufs& sb = on_side ? p.sb2 : p.sb;
    const SolveAssist* assist = !side ? nullptr : on_side ? &side->assist_side : &side->assist_main;
    CU(effective_ridge(Gi, d, d, rho, rho_relative, sb.rho, sq));
    if (bf16) SPCHK(ridge_core<float>(Ci, d, Gi, d, dh, d, nullptr, d, sb.rho, Wi, ldw, sb, status_dev, sq, assist));
    else SPCHK(ridge_core<double>(Ci, d, Gi, d, dh, d, nullptr, d, sb.rho, Wi, ldw, sb, status_dev, sq));
  }
  if (side) {
    CU(cudaEventRecord(side->join, side->stream));
    CU(cudaStreamWaitEvent(s, side->join, 0));
  }
  join_guard.armed = false;
  return SP_OK;
}

}  // extern "C"
