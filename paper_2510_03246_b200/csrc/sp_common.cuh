// Shared declarations of the libsp translation units (host-side launchers and small device helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/sp.h"

namespace sp {

// Device status word layout: status_dev[0] = code, [1] = failing index, [2] = aux, [3] = reserved.
__device__ __forceinline__ void report_status(int32_t* status, int32_t code, int32_t index, int32_t aux) {
  if (status == nullptr) return;
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = index;
    status[2] = aux;
  }
}

// ---- launch accounting and CUDA-event profiling (sp_profile.cu) ---------------------------------------------------
enum ProfKind : int {
  PK_GEMM_TC = 0, PK_GEMM_SIMT = 1, PK_SOLVE = 2, PK_FUSED_UPDATE = 3, PK_PREP_H = 4, PK_SCORES = 5, PK_TOPK = 6,
  PK_ELEMENTWISE = 7, PK_ALLOCATE = 8, PK_CHOL_DIAG = 9, PK_PANEL_APPLY = 10,
  PK_GEMM_TC_SHARED = 11,   // tensor-core GEMMs launched on a subset of the SM pairs, beside other work
  PK_CONDITIONAL = 12,      // tensor-core GEMMs queued under a SkipScope: whether they run is decided on the device, so
                            // neither their flops nor their time is attributed to the GEMM kinds
  PK_COUNT = 13
};
void count_launch(int n = 1);
// sp_set_reproducible: when on, every floating-point sum of the library is taken in an order fixed by the call's
// arguments (no product is cut along K, the triangular solves run on one stream), so equal inputs give equal bits.
bool reproducible_mode();
// sp_set_wait_budget: clock cycles a barrier wait of the tensor-core GEMM may take (0: the built-in default)
long long wait_budget_cycles();
// Device-side conditional work without a host round trip: while a SkipScope is alive on the calling host thread, the
// launchers that honour it (the kernels of the regularised solves, the tensor-core GEMM, the column gathers and
// scatters) pass its flag to their kernels, and every such kernel returns at once when the flag is non-zero at the
// time it starts.  The flag is written by an earlier kernel of the same stream order.  Scopes do not nest.
const int32_t* skip_flag();
struct SkipScope {
  explicit SkipScope(const int32_t* flag);
  ~SkipScope();
};
// Brackets the kernels launched during its lifetime with a CUDA event pair on `stream` when profiling is enabled.
// Scopes nest: only the outermost one records, so a phase scope absorbs the kernels launched inside it.
struct ProfScope {
  ProfScope(int kind, double flops, double bytes, cudaStream_t stream);
  ~ProfScope();
  int slot;
  cudaStream_t stream;
};

// One-time set-up per device (function attributes, device properties): run(fn) calls fn the first time it is reached
// with a given device current, under a lock, and remembers success per device; a process may drive several GPUs.
class PerDeviceOnce {
 public:
  template <typename F>
  cudaError_t run(F&& fn) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(mu_);
    if (done_[dev]) return cudaSuccess;
    e = fn();
    if (e == cudaSuccess) done_[dev] = true;
    return e;
  }
  static constexpr int kMaxDevices = 64;

 private:
  std::mutex mu_;
  bool done_[kMaxDevices] = {};
};
// Multiprocessor count of the current device (cached per device).
int sm_count();

__host__ __device__ __forceinline__ int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
__host__ __device__ __forceinline__ size_t align_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

inline size_t dtype_size(int32_t dt) { return dt == SP_BF16 ? 2 : (dt == SP_F64 ? 8 : 4); }

// A strided operand of the SIMT GEMM: element (i, k) lives at ptr[i * s0 + k * s1].
struct Operand {
  const void* ptr;
  int32_t dtype;
  int64_t s0, s1;
};

struct OutOperand {
  void* ptr;
  int32_t dtype;
  int64_t ld;
  // bf16 output of the tensor-core GEMM only: lo_off > 0 writes the result as two bf16 parts, bf16(v) at column j and
  // bf16(v - bf16(v)) at column lo_off + j of the same row, so that it can serve as a split operand of the next product
  int64_t lo_off = 0;
};

// C[M,N] (row-major) = alpha * sum_k A(i,k) B(k,j) + beta * Cin[i,j].  Cin may alias C or be another matrix of
// another dtype; beta == 0 never reads Cin.  lower_only skips tiles that lie strictly above the diagonal.
// acc64: accumulate in fp64 (else fp32).
cudaError_t gemm_simt(int64_t M, int64_t N, int64_t K, double alpha, Operand A, Operand B, double beta,
                      Operand Cin, OutOperand C, bool lower_only, bool acc64, cudaStream_t stream);

// tcgen05 path: bf16 operands, fp32 accumulation in tensor memory.
//   a_kmajor: A is stored [M, K] row-major (K contiguous) ; else [K, M] row-major (M contiguous).
//   b_kmajor: B is stored [N, K] row-major (K contiguous) ; else [K, N] row-major (N contiguous).
// Returns SP_ERR_UNSUPPORTED when alignment rules of the tensor maps are not met (the caller may then use gemm_simt).
struct TcOperand {
  const void* ptr;  // bf16
  int64_t ld;       // elements between consecutive rows of the stored matrix
  bool kmajor;
  int64_t kext = 0;   // extent of the stored matrix along K (0: the K of the call); reads beyond it return zero
  int64_t mnext = 0;  // extent along M (for A) or N (for B) (0: the M / N of the call)
};
// K segments: the contraction runs over nseg segments of K indices each; segment s reads A at K offset a_k[s] and
// M offset a_mn[s], B at K offset b_k[s] and N offset b_mn[s] (elements).  This is how split operands (an fp32 value
// held as a sum of bf16 parts stored side by side) are multiplied: one segment per kept product of parts.
constexpr int kTcMaxSegments = 6;
struct TcSegments {
  int32_t nseg = 1;
  int32_t a_k[kTcMaxSegments] = {0, 0, 0, 0, 0, 0}, a_mn[kTcMaxSegments] = {0, 0, 0, 0, 0, 0};
  int32_t b_k[kTcMaxSegments] = {0, 0, 0, 0, 0, 0}, b_mn[kTcMaxSegments] = {0, 0, 0, 0, 0, 0};
  // batched launches only: the plane of A / B the segment reads (see TcBatch)
  int32_t a_p[kTcMaxSegments] = {0, 0, 0, 0, 0, 0}, b_p[kTcMaxSegments] = {0, 0, 0, 0, 0, 0};
};
// Batched form: nb0 * nb1 independent products C_b = alpha A_b B_b (+ beta Cin_b) of the same shape in ONE launch.
// Operand X of product (b0, b1) starts at ptr + b0 * x_s0 + b1 * x_s1 (elements); this is how the per-head,
// per-sequence products of an attention module (head = a column slice of a token-major tensor, sequence = a row range)
// are issued together.  A and B may also consist of several planes (e.g. the hi and lo parts of a split operand, each
// a whole tensor, x_plane elements apart); a K segment then names the plane it reads.  Every stride times the element
// size must be a multiple of 16 bytes.  Not available together with lower_only or a cut along K.
struct TcBatch {
  int32_t nb0 = 1, nb1 = 1;
  int64_t a_s0 = 0, a_s1 = 0, b_s0 = 0, b_s1 = 0, c_s0 = 0, c_s1 = 0, cin_s0 = 0, cin_s1 = 0;
  int32_t a_planes = 1, b_planes = 1;
  int64_t a_plane = 0, b_plane = 0;
};
// K is the extent of ONE segment.  alg_flops >= 0 overrides the flop count recorded for profiling.  max_pairs > 0
// limits the launch to that many CTA pairs (SM pairs), leaving the other SMs to kernels of another stream.
sp_status gemm_tc(int64_t M, int64_t N, int64_t K, float alpha, TcOperand A, TcOperand B, float beta, Operand Cin,
                  OutOperand C, bool lower_only, int32_t* status_dev, cudaStream_t stream,
                  const TcSegments* segs = nullptr, double alg_flops = -1.0, int max_pairs = 0,
                  const TcBatch* batch = nullptr);
bool gemm_tc_supported(int64_t M, int64_t N, int64_t K, TcOperand A, TcOperand B);

// Dense symmetric positive definite solve in precision T (float or double), all on `stream`.
//   potrf: in-place lower Cholesky of the n x n matrix A (ld lda); the strict upper triangle is not referenced.
//   inv diag blocks are kept in `dinv` (n x NB row-major slabs) for the triangular solves.
struct CholWork {
  void* dinv;  // [ceil(n/NB) * NB * NB] elements of T
};
template <typename T>
cudaError_t potrf_lower(T* A, int64_t n, int64_t lda, T* dinv, int32_t* status_dev, cudaStream_t stream);
// X[m,n] <- X L^-T L^-1 (right solves with the factor of potrf_lower), i.e. X (L L^T)^-1.
template <typename T>
cudaError_t potrs_right(T* X, int64_t m, int64_t n, int64_t ldx, const T* L, int64_t ldl, const T* dinv,
                        cudaStream_t stream);
constexpr int kCholNB = 64;

// fp32 factorisation / solves with tensor-core trailing updates (sp_linalg_tc.cu).  Panels are kCholTcNB wide.
//   dinv: ceil(n / kCholTcNB) blocks of 2 * kCholTcNB^2 floats (inverse diagonal blocks and their transposes)
//   P   : bf16 [chol_tc_pad(n), 3 * chol_tc_pad(n)] — the factor below its diagonal blocks as three bf16 parts
//   Xs  : 2 x bf16 [m, 3 * kCholTcNB] — the current block column of the right-hand sides as three bf16 parts
constexpr int kCholTcNB = 128;
int64_t chol_tc_pad(int64_t n);
// Optional second stream (with three events) that carries the part of each step that the next step's first kernel
// does not wait for: the far part of a solve step's update; the panel and trailing update of a factorisation step.
struct SolveAssist {
  cudaStream_t stream;
  cudaEvent_t panel_done, rest_done[2];
  cudaEvent_t near_done;   // factorisation: the first two block columns of a step's trailing update have landed
  // Optional third stream of a factorisation: the far part of a step's trailing update (everything right of the first
  // two block columns), so that the next step's panel and near update do not queue behind it.
  cudaStream_t far_stream = nullptr;
  cudaEvent_t far_go = nullptr, far_done[2] = {nullptr, nullptr};
};
// dinv must have room for ceil(n / 128) + 1 pairs of 128 x 128 blocks (the last pair is scratch).
// m_extra > 0: A has m_extra more rows below row n (same lda), the right-hand sides B of a system X L^T = B; they
// are carried through the panels and trailing updates and hold X on return (P then needs n + m_extra rows).
sp_status potrf_lower_tc(float* A, int64_t n, int64_t lda, float* dinv, void* P, int32_t* status_dev,
                         cudaStream_t stream, const SolveAssist* assist = nullptr, int64_t m_extra = 0,
                         bool split_lookahead = false);   // lookahead kernel as two launches without a cluster
// Xs holds TWO buffers of [m, 3 * kCholTcNB] bf16.
// forward_done: X already holds the solution of the forward system (it rode along with the factorisation).
// Lf / ldl (optional): the fp32 factor potrf_lower_tc left in A; with it the backward sweep updates the next block
// column inside the panel kernel instead of by a GEMM of its own.
sp_status potrs_right_tc(float* X, int64_t m, int64_t n, int64_t ldx, const void* P, const float* dinv, void* Xs,
                         int32_t* status_dev, cudaStream_t stream, const SolveAssist* assist = nullptr,
                         bool forward_done = false, const float* Lf = nullptr, int64_t ldl = 0,
                         int64_t n_factor = 0);
// n_factor > n: the factor in P / dinv / Lf is that of a larger system of n_factor rows and the solve uses its leading
// n x n block, which is the factor of the system's leading block (n a multiple of kCholTcNB).

// `batch` independent systems of one size n (a multiple of kCholTcNB) with m right-hand sides each, every step one launch
// over all of them.  System b: A + b * a_bs = [n + m, n] fp32 (lower triangle of the matrix, then the right-hand sides
// B of X (L L^T) = B; on return they hold X), dinv + b * d_bs (room as for potrf_lower_tc), P = batch x
// [n + m, 3 n] bf16, Xs = batch x 2 x [m, 3 * kCholTcNB] bf16.
sp_status potrf_potrs_tc_batched(float* A, int64_t n, int64_t m, int batch, int64_t a_bs, float* dinv, int64_t d_bs,
                                 void* P, void* Xs, int32_t* status_dev, cudaStream_t stream);

// ---- elementwise / reduction launchers (sp_elementwise.cu) ------------------------------------------------------
cudaError_t convert_matrix(const void* src, int32_t sdt, int64_t lds, void* dst, int32_t ddt, int64_t ldd,
                           int64_t rows, int64_t cols, cudaStream_t stream);
cudaError_t symmetrize_lower(float* G, int64_t n, int64_t ld, cudaStream_t stream);
// dst[i, 0:cols] = bf16(src[i,:]) and dst[i, kpad:kpad+cols] = bf16(src - hi); padding columns are zero.
// dst is [rows, 2*kpad] bf16.
// row_idx != nullptr: row i of dst comes from row row_idx[i] of src.
cudaError_t split_bf16(const float* src, int64_t lds, const int32_t* row_idx, int64_t rows, int64_t cols, int64_t kpad,
                       void* dst, cudaStream_t stream);
// dst [rows, 3 * kpad] bf16: the hi, mid and lo parts of src side by side (an fp32 value as an exact sum of three bf16)
cudaError_t split3_bf16(const float* src, int64_t lds, int64_t rows, int64_t cols, int64_t kpad, void* dst,
                        cudaStream_t stream);
// dst[j, i] = (TD) src[i, j]
template <typename TD>
cudaError_t transpose_convert(const float* src, int64_t lds, int64_t rows, int64_t cols, TD* dst, int64_t ldd,
                              cudaStream_t stream);
int column_stats_row_blocks(int64_t T, int64_t C);
int score_row_blocks(int64_t rows, int64_t cols);
size_t wanda_scratch_doubles(int64_t rows, int64_t cols);
// weight statistics of the "-distribute" importances (sp_mask.cu); scratch: (148 * 8 + n_blocks) * 3 doubles
int weight_stats_parts(int64_t n_blocks, int64_t block_rows);
cudaError_t weight_stats(const void* W, int32_t dt, int64_t ld, int64_t rows, int64_t cols, int axis, int64_t group,
                         bool accumulate, double* stats, double* scratch, cudaStream_t stream);
cudaError_t distribute_importance(const double* head_stats, int n_heads, const double* fc_stats, int n_fc, int L,
                                  double rho, double gamma, double* I_attn, double* I_mlp, cudaStream_t stream);
// dst[i,j] = (T) G[i*ld + j] (+ rho on the diagonal) for the lower triangle; rho read from device (rho_dev[0]).
template <typename T>
cudaError_t load_spd(const float* G, int64_t ldg, int64_t n, const double* rho_dev, T* dst, int64_t ldd,
                     cudaStream_t stream);
// gathered version: dst[a,b] = G[idx[a], idx[b]] (+rho on diagonal), count read from host k.
template <typename T>
cudaError_t load_spd_gather(const float* G, int64_t ldg, const int32_t* idx, int64_t k, const double* rho_dev, T* dst,
                            int64_t ldd, cudaStream_t stream);
// dst [rows, kpad] (dense) = the first k columns of src followed by zero columns
cudaError_t copy_cols_padded(const float* src, int64_t lds, int64_t rows, int64_t k, int64_t kpad, float* dst,
                             cudaStream_t stream);
// dst[i, a] = (T) src[i, idx[a]]  (idx == nullptr: identity)
template <typename T>
cudaError_t gather_cols(const float* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k, T* dst,
                        int64_t ldd, cudaStream_t stream);
// dst[i, :] = src[idx[i], :]
cudaError_t gather_rows(const float* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t cols, float* dst,
                        int64_t ldd, cudaStream_t stream);
// dst (fp32, [rows, n]) = 0 ; dst[i, idx[a]] = src[i, a]
template <typename T>
cudaError_t scatter_cols(const T* src, int64_t lds, const int32_t* idx, int64_t rows, int64_t k, int64_t n,
                         float* dst, int64_t ldd, cudaStream_t stream);
// rho_out[0] = rho * trace(G)/n (relative) or rho
cudaError_t effective_ridge(const float* G, int64_t ldg, int64_t n, double rho, int rel, double* rho_out,
                            cudaStream_t stream);

struct UpdateArgs {
  float* Z;          // [T, n] in/out
  float* U;          // [T, n] in/out or null
  const float* z1;   // [T, ldk] compact on the kept channels
  const float* D;    // [T, ldk] compact: correction term of the a-update
  const float* gate; // [T, n] gate factor of a gated module (phi(z) = gate * z), or null: phi = ReLU
  int64_t ldk, k;    // leading dimension of the compact tensors, number of kept channels
  const int32_t* grp_base;   // per group of 8 channels: kept channels before the group
  const uint8_t* grp_mask;   // per group of 8 channels: bit q = channel 8 g + q is kept
  void* A_out;       // [T, n] storage dtype
  void* At_out = nullptr;  // bf16 [n, ldt]: A transposed (then A_out is not written)
  int64_t ldt = 0;
  void* Zb_out;      // [T, n] storage dtype copy of Z_new
  int32_t out_dtype;
  int64_t T, n;
  float alpha, beta;
  int32_t z_rule;
  double* partial;   // [blocks * 4] block partial sums: res_act, z_sq, a_sq, |z_new - z1|^2
  double* absA_part; // [row_blocks, n] partial column sums of |A|
  int32_t row_blocks;
  // At_out with its rows in "kept channels first" order: kept channel c goes to row (number of kept channels before
  // c), pruned channel c to row k + (number of pruned channels before c).
  int32_t at_kept_first = 0;
  // Both set (bf16 storage, ReLU, no dual variable, n % 4 == 0, At_out with at_kept_first; grid from
  // fused_update_next_grid): the update also writes what the next step reads, rows in the order of At_out, pitch ldt:
  // Zt_out [n, ldt] = bf16(Z_new)^T (the pruned channels' rows only when *zt_pruned_flag != 0 or the flag is null) and
  // Ht_out [k, ldt] = bf16(max(Z_new, 0))^T on the kept channels.  Zb_out is then not written.
  void* Zt_out = nullptr;
  void* Ht_out = nullptr;
  const int32_t* zt_pruned_flag = nullptr;
};
// grp_base / grp_mask of a u8 mask over n channels (see sp_elementwise.cu)
cudaError_t build_group_map(const uint8_t* mask, int64_t n, int32_t* grp_base, uint8_t* grp_mask, cudaStream_t stream);
// H[T, ldh] (compact on the k kept channels idx[0..k), ldh a multiple of 8) = storage(phi(Z) - U);
// phi(z) = gate * z when gate != nullptr, else ReLU.
// lo_off > 0 (bf16 storage, a multiple of 8, 2 * lo_off <= ldh): H is split into bf16 hi and lo parts, the hi part in
// columns [0, lo_off), the lo part in columns [lo_off, 2 * lo_off); columns k..lo_off-1 of both are zero.
cudaError_t launch_prep_h(const float* Z, const float* U, const float* gate, void* H, int32_t hdt, int64_t T,
                          int64_t n, int64_t ldh, int64_t k, const int32_t* idx, cudaStream_t stream,
                          int64_t lo_off = 0);
cudaError_t launch_fused_update(const UpdateArgs& a, cudaStream_t stream);
// Ht [k, ldt] bf16 = max(Z, 0)^T on the kept channels, rows in compact order (n % 4 == 0; ReLU, no dual variable): h of
// a step in the transposed layout in which the fused update leaves it for the next one.  Honours SkipScope.
cudaError_t launch_gather_ht(const float* Z, int64_t T, int64_t n, int64_t k, const int32_t* grp_base,
                             const uint8_t* grp_mask, void* Ht, int64_t ldt, cudaStream_t stream);
int fused_update_next_grid(int64_t T, int64_t n, int* row_blocks);
int fused_update_next_partial_rows(int row_blocks);   // rows of absA_part that this form of the update writes
int fused_update_next_row_cap(int64_t n);              // upper bound of the row blocks fused_update_next_grid returns
int64_t fused_update_next_max_blocks(int64_t n);       // ... and of its blocks
int fused_update_grid(int64_t T, int64_t n, int* row_blocks);
// out[j] (+)= sum_r part[r, j]
cudaError_t reduce_col_partials(const double* part, int32_t row_blocks, int64_t n, double* out, bool accumulate,
                                cudaStream_t stream);
// rep[field] (+)= sum of partial triples
cudaError_t reduce_report(const double* partial, int nblocks, sp_step_report* rep, bool accumulate, double alpha,
                          cudaStream_t stream);
// out[0] (+)= scale * sum of squares of a fp32 matrix; scratch: kSumsqBlocks doubles
constexpr int kSumsqBlocks = 592;
cudaError_t sumsq_accumulate(const float* x, int64_t ld, int64_t rows, int64_t cols, double scale, double* out,
                             bool accumulate, double* scratch, cudaStream_t stream);
// reused (device, may be null): non-zero when the recovery on the kept support reused the unrestricted factor
// scaled (device, may be null): non-zero when the pruned parts of G_A and R2 were obtained by scaling
cudaError_t init_report(sp_step_report* rep, const double* rho1, const double* rho2, double kept,
                        const int32_t* reused, const int32_t* scaled, cudaStream_t stream);
// relu + storage conversion for the init pass: A = phi(Z) -> storage dtype, and |A| column partials
// gate_io (gated modules): holds the gate pre-activation on entry and SiLU of it on return; A = gate * Z then
cudaError_t launch_init_act(const float* Z, float* gate_io, void* A_out, void* Zb_out, int32_t out_dtype, int64_t T,
                            int64_t n, double* absA_part, int32_t row_blocks, cudaStream_t stream);
cudaError_t column_stats(const void* X, int32_t dt, int64_t ld, int64_t T, int64_t C, double* rowstats,
                         double* scratch, cudaStream_t stream);

// ---- multi-head-attention auxiliary updates (sp_mha.cu); [pairs, T, T] tensors, pair = sequence * heads + head --------
// S <- softmax over each row (in place); causal: key u > query t gets 0; Sb: optional bf16 copy (plane > 0: hi and,
// `plane` elements further, lo parts)
cudaError_t mha_softmax_rows(float* S, int64_t pairs, int T, bool causal, void* Sb, int64_t plane, cudaStream_t stream);
// P <- P - eta_pair (-2 alpha G1 + 2 beta (P - Phi)); Pb: optional bf16 copy of the new P (hi / lo planes as above)
cudaError_t mha_p_update(float* P, const float* Phi, const float* G1, const float* eta, int64_t pairs, int T,
                         double alpha, double beta, void* Pb, int64_t plane, cudaStream_t stream);
// S (logits) <- dS = 2 beta Phi (E - rowsum(E Phi)), Phi = softmax(S), E = Phi - P; dSb: optional bf16 copy
cudaError_t mha_softmax_backward_rows(float* S, const float* P, int64_t pairs, int T, bool causal, double beta,
                                      void* dSb, cudaStream_t stream);
// per-pair step sizes from the squared norms of the [T, d_h] slices of x (and y): mode 0: 1 / (2 (alpha s + beta)),
// mode 1: eta_z / (2 alpha + beta s / d_h); sums: n_seq * H doubles of scratch
cudaError_t mha_step_sizes(const float* x, const float* y, int64_t ld, int64_t n_seq, int T, int d_h, int H, int mode,
                           double alpha, double beta, double eta_z, double* sums, float* eta, cudaStream_t stream);
// Z <- Z - eta_pair (G + 2 alpha (Z - T)) for Zq and Zk ([tokens, d] dense); Zqs / Zks: optional bf16 hi / lo planes
cudaError_t mha_z_update(float* Zq, float* Zk, const float* Gq, const float* Gk, const float* Tq, const float* Tk,
                         const float* eta, int64_t tokens, int d, int T, int d_h, double alpha, void* Zqs, void* Zks,
                         int64_t plane, cudaStream_t stream);
// A[n, n] (ld) = identity
cudaError_t set_identity(float* A, int64_t n, int64_t ld, cudaStream_t stream);
// dst[e] = bf16(x[e]), dst[plane + e] = bf16(x[e] - hi) (plane == 0: hi only)
cudaError_t split_planes(const float* x, int64_t total, void* dst, int64_t plane, cudaStream_t stream);

// ---- scores / allocation / selection (sp_mask.cu) -----------------------------------------------------------------
cudaError_t wanda_scores(int kind, int group, const float* W, int64_t rows, int64_t ldw, const float* colsq,
                         int64_t colsq_stride, const double* colabs, double inv_tokens, int64_t n_units,
                         float* scores, double* importance, double* scratch, cudaStream_t stream);
cudaError_t lemma1_scores_stream(const sp_mat& b, const sp_mat& c, const sp_mat& dd, const sp_mat& t, int group,
                                 int64_t n_units, float* scores, double* importance, double* relaxed, double r_layer,
                                 double* scratch, cudaStream_t stream);
// s_j = (cb_j + cc_j) / (2 cc_j) with cb_j = <T0[j,:], W1t[j,:]>, cc_j = <T0[j,:], W10[j,:]>, T0 = W10 G_X
cudaError_t lemma1_scores_gram(const float* T0, const float* W1t, const float* W10, int64_t n, int64_t d,
                               float* scores, double* importance, double* scratch, cudaStream_t stream);
cudaError_t allocate_sparsity(const double* I, const int64_t* n_units, int L, double rbar, double T, int mode,
                              double clip_hi, double* r_out, int64_t* k_out, cudaStream_t stream);
cudaError_t topk_select(const float* scores, int64_t n, int64_t k, uint8_t* mask, float* tau, int32_t* kept_idx,
                        cudaStream_t stream);
// kept_idx from an existing mask (ascending), count must equal k
// `batch` independent problems in one launch (one block each); k_list (device, may be nullptr) overrides k_all.
cudaError_t topk_select_batched(const float* scores, int64_t ld_scores, int64_t n, int64_t batch, int64_t k_all,
                                const int64_t* k_list, uint8_t* mask, int64_t ld_mask, float* tau, int32_t* kept_idx,
                                int64_t ld_idx, cudaStream_t stream, bool skip_negative = false);
// allocation for a grid of n_T temperatures in one launch: T_list (device), relative to mean |I| when T_relative;
// r_out / k_out are [n_T, L]
cudaError_t allocate_sparsity_grid(const double* I, const int64_t* n_units, int L, double rbar, const double* T_list,
                                   int n_T, bool T_relative, int mode, double clip_hi, double* r_out, int64_t* k_out,
                                   cudaStream_t stream);
// one threshold over the L x n scores (rows ld_scores apart): the K largest kept (ties: earlier layer, lower index),
// a layer left with fewer than min_keep units keeps its own min_keep best; counts_out[l] = kept units of layer l
size_t global_select_scratch_bytes(int64_t total, int L);
cudaError_t global_select(const float* scores, int64_t ld_scores, int64_t n, int L, int64_t K, int64_t min_keep,
                          uint8_t* mask, int64_t ld_mask, float* tau, int64_t* counts_out, void* scratch,
                          cudaStream_t stream);
cudaError_t mask_to_index(const uint8_t* mask, int64_t n, int32_t* kept_idx, cudaStream_t stream);
// reports SP_ERR_SHAPE (index = the number of kept units found) through the device status word when `mask` does not
// keep exactly k units; no-op without a status word
cudaError_t mask_count_check(const uint8_t* mask, int64_t n, int64_t k, int32_t* status, cudaStream_t stream);
// C[i, j] *= f^power for the rows x cols block at C (ld); f is read from the device (a float stored in an int32 slot)
cudaError_t scale_block(float* C, int64_t ld, int64_t rows, int64_t cols, const int32_t* f_bits, int power,
                        cudaStream_t stream);
// G[perm[i], perm[j]] = G[perm[j], perm[i]] = Gp[i, j] for i >= j (Gp: lower triangle in permuted order)
cudaError_t unpermute_gram(const float* Gp, const int32_t* perm, int64_t n, float* G, cudaStream_t stream);
// R[r, perm[j]] = Rp[r, j]
cudaError_t unpermute_cols(const float* Rp, const int32_t* perm, int64_t rows, int64_t n, float* R,
                           cudaStream_t stream);
// tag[1] = k when `valid`, else -1; tag[2] = bits of the float c; tag[4], tag[5] = size of the h buffer per token and
// token chunk with which h was written for the next step (0: none was written; its layout depends on both)
cudaError_t decay_tag_set(int32_t* tag, int64_t k, float c, bool valid, int64_t h_ld, int64_t h_chunk,
                          cudaStream_t stream);
// ready[0] = 1 when same[0] != 0 and the tag says that h was written for h_ld and h_chunk, else 0; ready[1] = 1 - ready[0]
cudaError_t h_next_ready(const int32_t* same, const int32_t* tag, int64_t h_ld, int64_t h_chunk, int32_t* ready,
                         cudaStream_t stream);
// R[perm[i], :] = Rp[i, :]
cudaError_t unpermute_rows(const float* Rp, const int32_t* perm, int64_t n, int64_t cols, float* R,
                           cudaStream_t stream);
// perm[0..n) = the kept channels of `mask` in ascending order followed by the pruned ones; count[0] = kept channels
cudaError_t mask_to_perm(const uint8_t* mask, int64_t n, int32_t* perm, int32_t* count, cudaStream_t stream);
// flags[0] = 1 when the kept channels of `mask` are not exactly perm[0..k) with count_old[0] == k; flags[1] = 1 - flags[0]
cudaError_t mask_changed(const uint8_t* mask, const int32_t* perm, const int32_t* count_old, int64_t k, int32_t* flags,
                         cudaStream_t stream);
cudaError_t zero_pruned(const uint8_t* mask, int group, float* W_rows, int64_t r_rows, int64_t r_cols, int64_t r_ld,
                        float* W_cols, int64_t c_rows, int64_t c_cols, int64_t c_ld, cudaStream_t stream);
// dst[i,:] = mask[i] ? src[i,:] : 0
cudaError_t mask_rows_copy(const uint8_t* mask, const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows,
                           int64_t cols, cudaStream_t stream);

}  // namespace sp
