/*
 * sp.h — C ABI of libsp: the per-module ADMM solve of structured SparseLLM / STRUPRUNE on one B200.
 *
 * What the library computes (paper: "StructPrune", arXiv 2510.03246):
 *   for one FFN module with input X = a_{l-1}^pre, up-projection W1 = W_l, down-projection W2 = W_{l+1},
 *   auxiliary variables Z = z_l, A = a_l and target Ypre = z_{l+1}^pre, minimise
 *       alpha |Ypre - W2 A|^2 + beta |A - phi(Z)|^2 + alpha |Z - W1 X|^2          (Appendix A.1, FFN objective)
 *   by alternating weight recovery W = z a^+ (Appendix A.1 "Reversely recovering the weight matrix"), the structured
 *   mask step (Lemma 1 / Section 3.4 scores, Lemma 2 / Algorithm 1 Step 2 allocation, Algorithm 1 Step 3 /
 *   Algorithm 3 threshold and M (.) W), the closed-form a-update and the z^(1)/z^(2) select (Algorithms 2 and 3).
 *
 * Conventions common to every call
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns every buffer; the
 *     library allocates no device memory.  Scratch comes from a caller workspace sized by sp_workspace_bytes().
 *   - All calls are asynchronous on the given CUDA stream (passed as void*, a cudaStream_t) and never synchronise.
 *   - Matrices are row-major with an explicit leading dimension `ld` (elements between consecutive rows).
 *     Calibration tensors are TOKEN-MAJOR: [tokens, channels] (the transpose of the paper's channel x token
 *     notation, i.e. the paper's matrix in column-major order).  Weights are [out, in].
 *   - Storage types: SP_BF16 or SP_F32 for activations (the "bf16 mode" / "fp32 mode"); accumulators, weights,
 *     Z and U are fp32; statistics and the allocation are fp64.
 *       bf16 mode: contractions run on the tensor cores with bf16 operands and fp32 accumulation; linear systems
 *                  are factorised in fp32.
 *       fp32 mode: contractions run in fp32 storage with fp64 accumulation; linear systems are factorised in fp64.
 *   - Return value: SP_OK or an error detected on the host before any launch (argument / shape / alignment /
 *     workspace errors).  Numerical failures found on the device (non-positive Cholesky pivot, a bounded wait that
 *     ran out) are written to the caller's `status_dev[4]` = {code, index, aux, 0}; nothing traps or spins forever.
 *   - Streams: a call is ordered on the caller's stream, but sp_admm_step, sp_admm_scores, sp_ridge_solve and
 *     sp_linear_refit also fork independent parts (the two weight recoveries, the panels and trailing updates of a
 *     factorisation, the z^(1) products) onto a few streams and events that the library creates once per device and
 *     joins back to the caller's stream with events before the call's results are used (also when a call returns an
 *     error after the fork).  That set is shared by all calls on a device: issue the calls of one device from one
 *     host thread at a time.  Nothing else persists inside the library.
 *   - Reproducibility: by default a product whose tile count leaves SMs idle is cut along K and its partial
 *     products add up in C in an order that is not fixed, and the backward triangular solve adds updates from two
 *     streams; fp32 results (accumulators, recovered weights, scores) can then differ in their last bits between two
 *     runs on equal inputs, and a mask can differ at scores that tie within that rounding.  sp_set_reproducible(1)
 *     switches both off (process-wide): every sum is then taken in an order fixed by the call's arguments and equal
 *     inputs give bit-identical outputs, at a few per cent of the step time.  The fp32 mode (fp64 accumulation on the
 *     CUDA cores, fp64 factorisation) and the score, statistics, report and selection kernels are reproducible either
 *     way.
 *   - Symmetric accumulators (Gram matrices) are stored as full squares; calls that update them keep the LOWER
 *     triangle (including the diagonal) authoritative.  sp_symmetrize() mirrors it to the upper triangle.
 */
#ifndef SP_H_
#define SP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SP_OK = 0,
  SP_ERR_INVALID_ARG = 1,
  SP_ERR_SHAPE = 2,
  SP_ERR_DTYPE = 3,
  SP_ERR_ALIGNMENT = 4,
  SP_ERR_WORKSPACE = 5,
  SP_ERR_NOT_SPD = 6,
  SP_ERR_TIMEOUT = 7,
  SP_ERR_CUDA = 8,
  SP_ERR_UNSUPPORTED = 9,
  SP_ERR_STATIC_LIMIT = 10
} sp_status;

typedef enum { SP_F32 = 0, SP_BF16 = 1, SP_F64 = 2 } sp_dtype;
typedef enum { SP_ACT_RELU = 0, SP_ACT_SWIGLU = 1 } sp_act_kind;
typedef enum { SP_Z_PAPER = 0, SP_Z_EXACT = 1 } sp_z_rule;
typedef enum { SP_SCORE_WANDA_L2 = 0, SP_SCORE_WANDA_L1 = 1, SP_SCORE_LEMMA1 = 2 } sp_score_kind;
typedef enum { SP_ALLOC_SOFTMAX = 0, SP_ALLOC_INVERSE = 1, SP_ALLOC_UNIFORM = 2 } sp_alloc_mode;
typedef enum { SP_WS_GRAM = 0, SP_WS_ADMM_STEP = 1, SP_WS_SCORES = 2, SP_WS_APPLY_MASK = 3, SP_WS_FFN_INIT = 4,
               SP_WS_LINEAR_REFIT = 5, SP_WS_GEMM = 6, SP_WS_RIDGE_SOLVE = 7, SP_WS_WEIGHT_STATS = 8,
               SP_WS_INPUT_INVERSE = 9 } sp_ws_op;

/* A row-major device matrix view. */
typedef struct {
  void* ptr;
  int32_t dtype; /* sp_dtype */
  int32_t reserved;
  int64_t rows, cols, ld;
} sp_mat;

/* Inputs of one FFN module (inputs of Algorithm 2, SparseLLM1). All read-only. */
typedef struct {
  sp_mat X;    /* [N, d]  module input a_{l-1}^pre, token-major, SP_BF16 or SP_F32 (selects the mode)          */
  sp_mat Ypre; /* [N, d]  pre-trained module output z_{l+1}^pre, same dtype as X (sp_ffn_init writes it)        */
  sp_mat W1_0; /* [n, d]  pre-trained up-projection, fp32 (used by sp_ffn_init and by the Lemma-1 score)         */
  sp_mat W2_0; /* [d, n]  pre-trained down-projection, fp32 (used by sp_ffn_init only)                           */
  int64_t d, n, N;
  int32_t act; /* sp_act_kind */
  int32_t reserved;
  sp_mat Wg_0; /* [n, d]  SP_ACT_SWIGLU only: pre-trained gate projection, fp32 (used by sp_ffn_init only)        */
} sp_ffn_module;

/* SP_ACT_SWIGLU is an extension: the paper's modules are ReLU FFNs.  The module is y = W2 (SiLU(Wg x) * (W1 x)); only
 * the "up" branch is split (Z ~ W1 X, A ~ g * Z) and the gate factor g = SiLU(Wg_0 X) is computed once by sp_ffn_init
 * into st->Gate and kept fixed, so phi(z) = g z is linear and every subproblem of the FFN objective keeps a closed
 * form: the recoveries and the a-update are those of the paper with phi(Z) = g Z, and the z-update is the single
 * quadratic minimiser Z = (beta g (A + U) + alpha z1) / (beta g^2 + alpha) (z_rule is not used).  The gate weights
 * are not recovered; the caller masks their rows with st->mask.  SP_SCORE_LEMMA1 is not available for this kind. */

/* ADMM state of one FFN module; every buffer is caller-owned device memory. */
typedef struct {
  float* Z;        /* [N, n] ld = n   auxiliary pre-activation z_l                                               */
  float* U;        /* [N, n] ld = n   scaled dual of a = phi(z), or NULL when dual_mode == 0                      */
  float* G_X;      /* [d, d]          X^T X (constant over the iterations)                                       */
  float* G_A;      /* [n, n]          A^T A of the current auxiliary activation                                  */
  float* R1;       /* [n, d]          Z^T X                                                                      */
  float* R2;       /* [d, n]          Ypre^T A                                                                   */
  double* absA;    /* [n]             sum over tokens of |A| per channel (Wanda l1 score)                         */
  float* W1;       /* [n, d]          out: masked recovered up-projection                                        */
  float* W2;       /* [d, n]          out: recovered down-projection on the kept support                          */
  float* scores;   /* [n]             out: unit scores of this step                                              */
  uint8_t* mask;   /* [n]             in/out: 1 = kept                                                           */
  double* importance; /* [1]          out: layer importance I_l = mean_j s_j                                      */
  float* Gate;     /* [N, n] ld = n   SP_ACT_SWIGLU only: g = SiLU(Wg_0 X), written by sp_ffn_init, then read-only   */
  float* G_X_inv;  /* [d, d]          optional cache (may be NULL): (G_X + rho1 I)^-1 written by
                                      sp_ffn_cache_input_inverse; read by sp_admm_step in bf16 mode                  */
  /* Optional (all three or none; used with bf16 storage, SP_ACT_RELU, dual_mode == 0, n % 4 == 0): the accumulators
   * of the new A in "kept channels first" order, kept from one step to the next.  A pruned channel has a zero row in
   * W1 and a zero column in W2, so its a = phi(z) and z_new = beta / (alpha + beta) * max(z, 0): from the second step
   * with an unchanged mask on, its row of A is c = beta / (alpha + beta) times the row of the step before.  With these
   * buffers sp_admm_step then obtains G_A[pruned, pruned] and R2[:, pruned] by scaling last step's values (c^2, c)
   * instead of contracting over the tokens again; the decision is taken on the device from decay_tag, which records
   * the channel order, k_keep and c of the last token pass.  G_A and R2 above are still written in channel order by
   * every step.  Whoever changes Z outside the library must set decay_tag[1] = -1; sp_ffn_init does. */
  float* G_A_perm;     /* [n, n]                                                                                     */
  float* R2_perm;      /* [d, n]                                                                                     */
  int32_t* decay_tag;  /* int32 [n + 8]                                                                              */
  /* Optional on top of the three above (both or none): R1 in the same way — Z of a pruned channel is c times its old
   * value too, so R1[pruned, :] is scaled, and only the kept rows are contracted.  For that the fused update writes the
   * bf16 copy of the new Z transposed with the kept channels first (instead of a row-major copy), and from the same
   * registers h = max(Z_new, 0) of the kept channels into H_next: the a-update of the NEXT step starts from it and makes
   * no gather pass over Z while the mask stays, so that Z is read once and written once per step.  Used when N % 8 == 0.
   * Layout of H_next (the library's own; it depends on the token chunk): for the chunk of Tc tokens that starts at
   * token t0, the k_keep x Tc block h^T (kept channels in ascending order, tokens contiguous) at element
   * t0 * H_next_ld. */
  float* R1_perm;      /* [n, d]                                                                                     */
  void* H_next;        /* N * H_next_ld bf16 elements                                                                */
  int64_t H_next_ld;   /* a multiple of 8, at least ceil8(k_keep); smaller: R1_perm / H_next are not used             */
} sp_ffn_state;

typedef struct {
  double alpha, beta;      /* penalty weights of the FFN objective (Appendix A.1)                                  */
  double rho;              /* Tikhonov term of the weight recovery: W = R (G + rho_eff I)^-1                       */
  int32_t rho_relative;    /* 1: rho_eff = rho * trace(G)/dim(G);  0: rho_eff = rho                                */
  int32_t z_rule;          /* sp_z_rule: literal select of Algorithms 2/3, or exact scalar minimiser               */
  int32_t dual_mode;       /* 0: paper's penalty form; 1: scaled dual U on a = phi(z) (an extension of the paper)  */
  int32_t score_kind;      /* sp_score_kind                                                                       */
  int64_t k_keep;          /* units kept in this module (from sp_allocate_sparsity)                                */
  int32_t reselect_mask;   /* 1: recompute the top-k mask from this step's scores; 0: keep st->mask, which must keep
                              exactly k_keep units (else SP_ERR_SHAPE through status_dev, index = units it keeps)   */
  int32_t refit;           /* 1: recovery solver on the kept support (Algorithm 2); 0: plain M (.) W               */
  int64_t token_chunk;     /* tokens per streamed chunk (0 = library default)                                      */
  int32_t compute_objective; /* 1: also report alpha|Ypre-W2A|^2 (one more product per token chunk)                 */
  int32_t skip_scores;     /* 1 (needs reselect_mask = 0 and refit = 1): the mask is fixed, so the unrestricted
                              recovery W2~ and the unit scores, which only serve the mask selection, are not computed;
                              st->scores and st->importance keep their previous values                              */
} sp_admm_params;

/* Device-side report of one step (all double). */
typedef struct {
  double res_act;   /* |A - phi(Z_new)|^2                                                                         */
  double res_out;   /* alpha |Ypre - W2 A|^2   (NaN unless compute_objective)                                      */
  double res_in;    /* alpha |Z_new - W1 X|^2                                                                      */
  double z_sq;      /* |Z_new|^2                                                                                  */
  double a_sq;      /* |A|^2                                                                                      */
  double rho1_eff, rho2_eff; /* ridge terms actually used                                                         */
  double kept;      /* number of kept units                                                                       */
  double factor_reused; /* 1: the recovery on the kept support was one backward sweep with the leading block of the
                           unrestricted factor (the new mask kept the channels of the previous one); else 0         */
  double pruned_scaled; /* 1: G_A[pruned, pruned] and R2[:, pruned] were obtained by scaling last step's values
                           (see sp_ffn_state.G_A_perm); else 0                                                      */
} sp_step_report;

/* Inputs of sp_struct_scores; only the fields of the chosen kind are read. */
typedef struct {
  sp_mat W;              /* WANDA kinds: fp32 weight [out, n_units*group] whose COLUMNS belong to the units         */
  const float* colsq;    /* WANDA_L2: sum_t a_jt^2 per column, element j at colsq[j*colsq_stride] (e.g. diag of G)  */
  int64_t colsq_stride;
  const double* colabs;  /* WANDA_L1: sum_t |a_jt| per column                                                       */
  double inv_tokens;     /* WANDA_L1: 1/N                                                                           */
  sp_mat b, c, dd, t;    /* LEMMA1: token-major [N, n_units*group] streams (fp32 or bf16), see Lemma 1              */
} sp_score_inputs;

/* ---------------------------------------------------------------------------------------------------------------
 * sp_gram_accumulate — Gram and cross-product accumulation over one chunk of calibration tokens.
 * Paper: these are the two products the weight recovery W = z a^+ = (z a^T)(a a^T)^-1 needs (Appendix A.1,
 * "Reversely recovering the weight matrix"; Algorithm 3 first line of the step).
 *   G[C,C] += Xc^T Xc (lower triangle authoritative),  R[Rr,C] += Yc^T Xc (skipped when Yc == NULL),
 *   rowstats[c,0] += sum_t |Xc[t,c]|, rowstats[c,1] += sum_t Xc[t,c]^2 (skipped when NULL; fp64).
 * Xc: [T, C], Yc: [T, Rr], same dtype (SP_BF16 or SP_F32).  G, R: fp32, ldg >= C, ldr >= C.
 * Workspace: sp_workspace_bytes(SP_WS_GRAM, C, Rr, T, 0, dtype).  status_dev may be NULL.
 * Errors: SP_ERR_INVALID_ARG (null pointers), SP_ERR_SHAPE (row counts differ, ld too small), SP_ERR_DTYPE,
 *         SP_ERR_WORKSPACE.
 */
sp_status sp_gram_accumulate(const sp_mat* Xc, const sp_mat* Yc, float* G, int64_t ldg, float* R, int64_t ldr,
                             double* rowstats, int32_t* status_dev, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_ffn_init — initialisation of Algorithm 2 (SparseLLM1): z = z^pre = X W1_0^T, a = a^pre = phi(z^pre),
 * Ypre = a^pre W2_0^T (written to m->Ypre), and the accumulators G_X, G_A, R1, R2, absA of that state.
 * U (if not NULL) is cleared.  Workspace: sp_workspace_bytes(SP_WS_FFN_INIT, d, n, N, token_chunk, dtype).
 */
sp_status sp_ffn_init(const sp_ffn_module* m, sp_ffn_state* st, int64_t token_chunk, int32_t* status_dev,
                      void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_ffn_cache_input_inverse — the cached pseudo-inverse of the module input of Algorithm 2 (SparseLLM1, "pre-compute
 * and cache a_{l-1}^+"): the input never changes over the iterations, so neither does G_X + rho1 I.  Writes
 * st->G_X_inv = (G_X + rho1 I)^-1 (fp32 [d, d], factorised and inverted in fp64) after sp_ffn_init.  With it,
 * sp_admm_step (bf16 mode) recovers W1~ = R1 (G_X + rho1 I)^-1 as ONE tensor-core product with both operands carried
 * as three bf16 parts instead of a factorisation and two triangular sweeps per step.  rho / rho_relative must be the
 * values later passed in sp_admm_params (the caller's responsibility; a step with st->G_X_inv == NULL, and every step
 * in fp32 mode, solves the system itself).  Workspace: sp_workspace_bytes(SP_WS_INPUT_INVERSE, d, 0, 0, 0, 0).
 * Errors: SP_ERR_INVALID_ARG (null G_X / G_X_inv, rho < 0), SP_ERR_SHAPE, SP_ERR_WORKSPACE, SP_ERR_ALIGNMENT.
 */
sp_status sp_ffn_cache_input_inverse(const sp_ffn_module* m, sp_ffn_state* st, double rho, int32_t rho_relative,
                                     int32_t* status_dev, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_admm_step — one outer step of Algorithm 2 (SparseLLM1) in the per-step order of Algorithm 3 (GSPO):
 *   1. W1~ = R1 (G_X + rho1 I)^-1, W2~ = R2 (G_A + rho2 I)^-1        (weight recovery, Appendix A.1)
 *   2. unit scores (p->score_kind) and layer importance              (Lemma 1 / Section 3.4 / Algorithm 1 Step 3)
 *   3. top-k mask with k = p->k_keep if p->reselect_mask             (Algorithm 3 threshold; exactly k kept)
 *   4. W1 = diag(M) W1~;  W2[:,S] = R2[:,S] (G_A[S,S] + rho2 I)^-1   (recovery on the kept support, or M (.) W2~)
 *   5. per token chunk: A = h + (Ypre - h W2^T)(gamma I + W2 W2^T)^-1 W2 with h = phi(Z) - U, gamma = beta/alpha,
 *      which equals a_l = (alpha W2^T W2 + beta I)^-1 (alpha W2^T Ypre + beta h) of Appendix A.1;
 *      z^(1) = X W1^T, z^(2) = (beta (A+U) + alpha z^(1))/(alpha+beta); select; U += A - phi(Z_new);
 *      G_A, R1, R2, absA are rebuilt from the new A and Z.
 * Steps 1 and 4 share a factorisation when they can (bf16 storage, refit): the system of step 1 is factorised with
 * the channels that st->mask kept BEFORE the call in front, so the leading block of its factor is the factor of
 * G_A[S',S'] + rho2 I for that support S'.  When the mask of step 3 keeps exactly those channels, step 4 is a backward
 * sweep with that block (rep->factor_reused = 1); otherwise the restricted system is factorised.  The decision is
 * taken on the device; both ways give the same restricted ridge solution up to rounding.
 * In/out: st (Z, U, accumulators, mask); out: st->W1, st->W2, st->scores, st->importance, *rep_dev.
 * rep_dev and status_dev are device pointers (status_dev: int32[4], must be zeroed by the caller beforehand).
 * Workspace: sp_workspace_bytes(SP_WS_ADMM_STEP, d, n, N, token_chunk, dtype).
 * Errors: SP_ERR_INVALID_ARG, SP_ERR_SHAPE (k_keep outside [1, n], N/d/n mismatch), SP_ERR_DTYPE, SP_ERR_WORKSPACE.
 */
sp_status sp_admm_step(const sp_ffn_module* m, sp_ffn_state* st, const sp_admm_params* p, sp_step_report* rep_dev,
                       int32_t* status_dev, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_admm_scores — parts 1 and 2 of sp_admm_step alone: the unrestricted recovery the scores read (W2~; W1~ as well
 * for SP_SCORE_LEMMA1) and the unit scores and layer importance of the module's current state.  Writes st->scores
 * and st->importance; st->W1, st->W2, st->mask, Z, U and the accumulators are left as they are.
 * Paper: Appendix B, Algorithm 3 (GSPO) collects the scores of ALL layers before one global threshold decides every
 * mask; a lock-step run calls this for every module, selects over the concatenated scores (sp_apply_mask), and then
 * finishes the iteration of each module with sp_admm_step(reselect_mask = 0, skip_scores = 1).
 * p->k_keep is ignored; p->skip_scores must be 0.  Workspace and errors as sp_admm_step.
 */
sp_status sp_admm_scores(const sp_ffn_module* m, sp_ffn_state* st, const sp_admm_params* p, int32_t* status_dev,
                         void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_struct_scores — per-unit importance scores and the layer importance I = mean over units.
 *   SP_SCORE_WANDA_L2 (Section 3.4, Eq. "wanda"): s_u = sqrt( sum_{j in unit u} |W[:,j]|_2^2 * colsq_j )
 *   SP_SCORE_WANDA_L1 (Algorithm 1, Step 3):       s_u = sum_{j in unit u} |W[:,j]|_1 * colabs_j * inv_tokens
 *   SP_SCORE_LEMMA1   (Lemma 1, Eq. 3; inner products over tokens):
 *        s_u = sum_{j in u}(<c_j,b_j> + <d_j,t_j>) / sum_{j in u}(|c_j|^2 + |d_j|^2)
 * group = rows/columns per unit (1 = channel, d_head = attention head).
 * scores: fp32 [n_units]; layer_importance: fp64 [1]; relaxed_mask (optional, fp64 [n_units], LEMMA1 only):
 *   M_u = s_u - (1/e_u)(sum_k s_k - r_layer n_units)/sum_k(1/e_k), e_u the denominator of s_u (Appendix B, Eq. Mlj).
 * Workspace: sp_workspace_bytes(SP_WS_SCORES, n_units*group, 0, N, 0, dtype).
 */
sp_status sp_struct_scores(int32_t kind, int32_t group, const sp_score_inputs* in, int64_t n_units, float* scores,
                           double* layer_importance, double* relaxed_mask, double r_layer, void* ws, size_t ws_bytes,
                           void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_struct_scores_static — the two Wanda kinds of sp_struct_scores with NO workspace argument and no allocation.
 * The paper has no counterpart; this is a packaging variant of the call above.
 * Who needs it: a caller that owns no spare device memory and cannot obtain any — for example a service whose device
 * memory was carved up once at start-up, or code that runs between other asynchronous work and must not stall the
 * whole device the way an allocation call does.  Such a caller passes only the inputs and the outputs; the partial
 * column sums go to a fixed array of 2 MiB that is part of the library image (every GPU that loads libsp.so holds
 * it until the process ends).
 * Limits: n_units*group <= SP_STATIC_SCORES_MAX_COLS, and the partial sums must fit the array; anything larger
 * returns SP_ERR_STATIC_LIMIT before any launch (use sp_struct_scores with a workspace instead).  kind must be
 * SP_SCORE_WANDA_L2 or SP_SCORE_WANDA_L1 (else SP_ERR_UNSUPPORTED).  Other argument errors as sp_struct_scores.
 * Results are the same as sp_struct_scores gives for the same inputs (same kernels, same reduction order).
 * Set-up: the first call on each device looks up the device address of the array (one runtime query, with that device
 * current); make that first call outside any stream capture.
 * Sharing: all calls on one device use the same array.  Calls on the same stream are ordered and safe; two calls that
 * may overlap on the GPU (different streams without an ordering between them) race on it.  The array keeps the last
 * call's partial sums; no call reads a partial sum it did not write itself, and the few arrival counters at its end,
 * which must start at zero, are cleared on the stream at the start of every call.
 * The call itself performs no device or host allocation and calls no allocating library routine.
 */
#define SP_STATIC_SCORES_MAX_COLS 32768
sp_status sp_struct_scores_static(int32_t kind, int32_t group, const sp_score_inputs* in, int64_t n_units,
                                  float* scores, double* layer_importance, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_allocate_sparsity — softmax-form sparsity allocation across L layers (Lemma 2; Algorithm 1, Step 2).
 *   SOFTMAX: w = softmax(-I/T); r = rbar L w; clip to [0, clip_hi]; if no entry hit clip_hi: rescale to mean rbar,
 *            clip again.  INVERSE: r = clip(rbar L (1-w)/sum(1-w)) (Algorithm "-distribute", Step 2).  UNIFORM: rbar.
 *   r_l is the fraction PRUNED; k_keep_out[l] = n_units[l] - floor(r_l n_units[l] + 0.5).  All fp64 / int64, device.
 * Errors: SP_ERR_INVALID_ARG (null, T <= 0, rbar outside [0,1]), SP_ERR_SHAPE (L < 1 or L > 65536).
 */
sp_status sp_allocate_sparsity(const double* I, const int64_t* n_units, int32_t L, double rbar, double T, int32_t mode,
                               double clip_hi, double* r_out, int64_t* k_keep_out, void* stream);

/* sp_allocate_sparsity_grid — the allocation above for a whole grid of temperatures in one launch (the outer loop of
 * Algorithm 1 runs Step 2 once per temperature of its search grid).  T_list: fp64 [n_T] on the device; T_relative != 0:
 * entry T_list[g] is given relative to the magnitude of the importances, T = T_list[g] * mean_l |I_l| (computed on the
 * device; Section 4 scales the temperature to the importance scores).  r_out, k_keep_out: [n_T, L], row g for T_list[g].
 * Errors as sp_allocate_sparsity, plus SP_ERR_SHAPE for n_T outside [1, 65535]. */
sp_status sp_allocate_sparsity_grid(const double* I, const int64_t* n_units, int32_t L, double rbar, const double* T_list,
                                    int32_t n_T, int32_t T_relative, int32_t mode, double clip_hi, double* r_out,
                                    int64_t* k_keep_out, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_apply_mask — top-k selection and M (.) W (Algorithm 1 Step 3; Algorithm 3 threshold and mask lines).
 * Keeps exactly k_keep units: the k largest scores, equal scores resolved toward the lower index, NaN lowest.
 * mask_out: u8 [n_units] (1 = kept); tau_out (optional): the k-th largest score; kept_idx_out (optional): int32
 * [k_keep] ascending indices of kept units.  W_rows (optional, fp32 [n_units*group, cols]): rows of pruned units are
 * zeroed.  W_cols (optional, fp32 [rows, n_units*group]): columns of pruned units are zeroed.
 * Errors: SP_ERR_SHAPE (k_keep outside [0, n_units], matrix sizes do not match n_units*group).
 */
sp_status sp_apply_mask(const float* scores, int64_t n_units, int64_t k_keep, int32_t group, uint8_t* mask_out,
                        float* tau_out, int32_t* kept_idx_out, const sp_mat* W_rows, const sp_mat* W_cols, void* ws,
                        size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_apply_mask_batched — the top-k selection of Algorithm 1 Step 3 for all L layers of a model in one launch.
 * Layer l has its own score vector scores + l * ld_scores (n_units each) and its own kept count k_keep[l], read on the
 * DEVICE (the integer counts sp_allocate_sparsity wrote can be passed on without a host round trip); counts outside
 * [0, n_units] are clamped.  Same selection rule as sp_apply_mask.  Outputs per layer: mask_out + l * ld_mask (u8
 * [n_units]); tau_out[l] (optional); kept_idx_out + l * ld_idx (optional, int32, the first k_keep[l] entries are
 * written).  No weights are touched.  All pointers are device pointers.
 * Errors: SP_ERR_INVALID_ARG (null scores / k_keep / mask_out), SP_ERR_SHAPE (negative sizes, a leading dimension
 * smaller than n_units).
 */
sp_status sp_apply_mask_batched(const float* scores, int64_t ld_scores, int64_t n_units, int32_t L,
                                const int64_t* k_keep, uint8_t* mask_out, int64_t ld_mask, float* tau_out,
                                int32_t* kept_idx_out, int64_t ld_idx, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_apply_mask_global — the threshold step of Appendix B, Algorithm 3 (GSPO) over all L layers at once: the scores of
 * all layers (row l at scores + l * ld_scores, n_units each) are collected, K = floor(keep_fraction * n_units * L),
 * and the units holding the K largest scores are kept: one threshold for the whole model.  Exactly K units are kept
 * (ties: the earlier layer, then the lower index; NaN lowest), unless min_keep > 0: a layer the threshold leaves with
 * fewer than min_keep units keeps its own min_keep best instead (as printed the algorithm can empty a layer).
 * mask_out: u8, row l at mask_out + l * ld_mask; tau_out (optional): the K-th largest score; kept_out: int64 [L] kept
 * units per layer after the repair (device).  The select runs on many CTAs (four histogram passes over the keys), so
 * L * n_units is not limited by one CTA's shared memory; up to 47104 keys in contiguous rows are selected by one CTA
 * instead, which is faster there (same result).  Workspace: sp_apply_mask_global_bytes(n_units, L).
 * Errors: SP_ERR_INVALID_ARG (null pointers, keep_fraction outside [0, 1]), SP_ERR_SHAPE, SP_ERR_WORKSPACE,
 * SP_ERR_ALIGNMENT (workspace not 256-byte aligned). */
sp_status sp_apply_mask_global(const float* scores, int64_t ld_scores, int64_t n_units, int32_t L, double keep_fraction,
                               int64_t min_keep, uint8_t* mask_out, int64_t ld_mask, float* tau_out,
                               int64_t* kept_out, void* ws, size_t ws_bytes, void* stream);
size_t sp_apply_mask_global_bytes(int64_t n_units, int32_t L);

/* sp_objective_accumulate — Step 5 of Algorithm 1: loss_dev[0] (+)= L_l = res_out + beta * res_act + res_in of a step
 * report (the FFN objective of Appendix A.1 after that step; needs compute_objective).  All pointers on the device. */
sp_status sp_objective_accumulate(const sp_step_report* rep_dev, double beta, double* loss_dev, int32_t accumulate,
                                  void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_weight_stats, sp_distribute_importance — the weight-statistic importances of the "-distribute" variant of
 * Algorithm 1 (its Step 1): per attention head |W_h|_1 + 0.1 Var(W_h) + 0.01 |W_h|_2, per MLP matrix
 * |W_m|_1 + 0.05 Var(W_m), times the depth weight gamma^l (layers counted from 1) and, for attention, the
 * attention/MLP ratio rho.  Step 2 of that algorithm is sp_allocate_sparsity with SP_ALLOC_INVERSE.
 *
 * sp_weight_stats: sums over slices of one weight matrix W (fp32 or bf16, [rows, cols], device).
 *   axis = 0: block b is rows [b*group, (b+1)*group) (all columns);  axis = 1: block b is columns [b*group, ...)
 *   (all rows);  group = 0: the whole matrix is one block.  rows (axis 0) / cols (axis 1) must be a multiple of group.
 *   stats: fp64 [n_blocks, 4] on the device = {sum |w|, sum w, sum w^2, number of entries}; accumulate != 0 adds to
 *   what it holds, so the slices of one head in W_Q, W_K, W_V (axis 0) and W_O (axis 1) add up to that head's sums.
 *   Workspace: sp_workspace_bytes(SP_WS_WEIGHT_STATS, n_blocks, 0, 0, 0, 0).  Deterministic (fixed summation order).
 *   Errors: SP_ERR_INVALID_ARG (null pointers, axis not 0/1), SP_ERR_DTYPE, SP_ERR_SHAPE (group does not divide the
 *   extent, ld < cols), SP_ERR_WORKSPACE.
 * sp_distribute_importance: head_stats fp64 [L, n_heads, 4] and fc_stats fp64 [L, n_fc, 4] as written above (either
 *   may be NULL, then its output is not written); I_attn, I_mlp fp64 [L] on the device.  The variance is the
 *   population variance sum w^2 / c - (sum w / c)^2 over the c entries, the l2 norm sqrt(sum w^2).
 */
sp_status sp_weight_stats(const sp_mat* W, int32_t axis, int64_t group, int32_t accumulate, double* stats, void* ws,
                          size_t ws_bytes, void* stream);
sp_status sp_distribute_importance(const double* head_stats, int32_t n_heads, const double* fc_stats, int32_t n_fc,
                                   int32_t L, double rho, double gamma, double* I_attn, double* I_mlp, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_mha_init, sp_mha_step — auxiliary-variable updates of one attention module under the paper's second objective
 * (Appendix A, "Computation on Multi-Head Attention layers", Method 2; Algorithm 2, SparseLLM2), weights held fixed.
 *
 * Module (paper, per sequence of T tokens and per head i of width d_h = d / n_heads, tokens as columns):
 *   Q = W_Q X, K = W_K X, V = W_V X;  S_i = Q_i^T K_i / sqrt(d_h);  P_i = softmax over the keys of each row of S_i;
 *   head_i = V_i P_i^T;  a_attn = Concat_i head_i;  z_{l+1}^pre = W_O a_attn.
 * Storage is token-major: X, Ypre, Zq, Zk, Aattn are [n_seq * T, d]; head i owns columns [i d_h, (i+1) d_h);
 * P is [n_seq, n_heads, T, T] (row = query, column = key), fp32.
 * Reading of Method 2 (the section prints inconsistent shapes): the auxiliary output z_l is the pair (Zq, Zk) with
 * Zq ~ W_Q X and Zk ~ W_K X ("separate constraints for each projection"), a_l is P, a_attn_l the concatenated heads:
 *   alpha |Ypre - W_O Aattn|^2 + alpha |Aattn - Concat_i V_i P_i^T|^2 + beta |P - softmax(S(Zq, Zk))|^2
 *   + alpha |Zq - W_Q X|^2 + alpha |Zk - W_K X|^2.
 * sp_mha_init writes the forward definition: Zq, Zk, P, Aattn and Ypre = Aattn W_O^T (the pre-trained state).
 * sp_mha_step, in the order of Algorithm 2:
 *   Eq. (85)  a_steps gradient steps on every P_i of alpha |Aattn_i - V_i P_i^T|^2 + beta |P_i - softmax(S_i)|^2 with
 *             the step 1 / (2 (alpha |V_i|_F^2 + beta));
 *   Eq. (86)  Aattn = (W_O^T W_O + I)^-1 (W_O^T Ypre + Concat_i V_i P_i^T)   (closed-form minimiser);
 *   Eq. (87)  z_steps joint gradient steps on (Zq_i, Zk_i) of beta |P_i - softmax(S_i)|^2 + alpha |Zq_i - (W_Q X)_i|^2
 *             + alpha |Zk_i - (W_K X)_i|^2 through the softmax, with the step
 *             eta_z / (2 alpha + beta (|Zq_i|_F^2 + |Zk_i|_F^2) / d_h) recomputed before every step.
 * The elementwise "if z < 0" select that Algorithm 2 repeats for this module belongs to the ReLU module; it is not
 * applied.  causal != 0 masks keys after the query.  The weights (already masked by the caller: pruned heads have zero
 * rows in W_Q, W_K, W_V and zero columns in W_O) are read only; their recovery from the updated variables uses
 * sp_gram_accumulate / sp_ridge_solve / sp_linear_refit.
 * bf16 mode (X bf16): all contractions are batched tensor-core products (one launch for all heads and sequences of a
 * chunk), operands whose rounding matters carried as bf16 hi + lo parts; needs d_h % 8 == 0 and T % 8 == 0
 * (SP_ERR_ALIGNMENT otherwise).  fp32 mode: fp32 operands, fp64 accumulation.
 * seq_chunk sequences are processed at a time (0 = 1); workspace: sp_mha_workspace_bytes(d, n_heads, T, n_seq,
 * seq_chunk, dtype of X).  Errors: SP_ERR_INVALID_ARG (null pointers, alpha / beta <= 0, eta_z outside (0, 1],
 * negative counts), SP_ERR_SHAPE (sizes that do not match d, n_heads, T, n_seq; leading dimensions other than d),
 * SP_ERR_DTYPE, SP_ERR_ALIGNMENT, SP_ERR_WORKSPACE.
 */
typedef struct {
  sp_mat X;     /* [n_seq * T, d] module input, SP_BF16 or SP_F32 (selects the mode), ld = d                      */
  sp_mat Ypre;  /* [n_seq * T, d] pre-trained module output, same dtype (sp_mha_init writes it), ld = d             */
  sp_mat Wq, Wk, Wv, Wo;   /* [d, d] fp32, [out, in], ld = d                                                       */
  int64_t d, n_heads, T, n_seq;
} sp_mha_module;

typedef struct {
  float* Zq;     /* [n_seq * T, d]             auxiliary output of the query projection                            */
  float* Zk;     /* [n_seq * T, d]             auxiliary output of the key projection                              */
  float* P;      /* [n_seq, n_heads, T, T]     auxiliary attention probabilities a_l                               */
  float* Aattn;  /* [n_seq * T, d]             auxiliary concatenated head outputs a_attn_l                        */
  /* Optional accumulators over all tokens (all five or none; NULL = not computed), rebuilt by sp_mha_init and by
   * every sp_mha_step from the variables it leaves, for the weight recoveries W = z a^+ of the next outer iteration
   * ("do for W_Q, W_K, W_V, W_O separately"):  W_Q = R_Q (G_X + rho I)^-1, W_K = R_K (G_X + rho I)^-1 by
   * sp_ridge_solve;  W_O[:, S] = R_O[:, S] (G_attn[S,S] + rho I)^-1 on the columns of the kept heads by
   * sp_linear_refit.  fp32 [d, d] each, Gram matrices as full squares. */
  float* G_X;    /* X^T X                                                                                          */
  float* R_Q;    /* Zq^T X                                                                                         */
  float* R_K;    /* Zk^T X                                                                                         */
  float* G_attn; /* Aattn^T Aattn                                                                                  */
  float* R_O;    /* Ypre^T Aattn                                                                                   */
} sp_mha_state;

typedef struct {
  double alpha, beta;
  int32_t a_steps, z_steps;  /* gradient steps of Eq. (85) and Eq. (87)                                            */
  double eta_z;              /* relative step of Eq. (87), in (0, 1]                                               */
  int32_t causal;
  int32_t reserved;
  int64_t seq_chunk;
} sp_mha_params;

sp_status sp_mha_init(const sp_mha_module* m, sp_mha_state* st, int32_t causal, int64_t seq_chunk, int32_t* status_dev,
                      void* ws, size_t ws_bytes, void* stream);
sp_status sp_mha_step(const sp_mha_module* m, sp_mha_state* st, const sp_mha_params* p, int32_t* status_dev, void* ws,
                      size_t ws_bytes, void* stream);
size_t sp_mha_workspace_bytes(int64_t d, int64_t n_heads, int64_t T, int64_t n_seq, int64_t seq_chunk, int32_t dtype);

/* ---------------------------------------------------------------------------------------------------------------
 * sp_mha_value_refit — recovery of W_V from the auxiliary variables of an attention module.
 * Paper: Appendix A, Method 2, "Recovering weight matrices" (W = z a^+) applied to the second term of the objective,
 * alpha |a_attn - Concat_i(W_V,i a_i)|^2; Algorithm 2 runs the recovery "for W_Q, W_K, W_V, W_O separately".
 * With a_l the attention probabilities P the term ties head i's columns of Aattn to W_V through
 *   Aattn_i = (P_i X) W_V,i^T      per sequence (token-major: [T, d_h] = [T, T] [T, d] [d, d_h]),
 * so the regressors of head i are R_i = P_i X and its ridge least-squares solution over all sequences s is
 *   W_V,i = (sum_s Aattn_i,s^T R_i,s) (sum_s R_i,s^T R_i,s + rho_i I)^-1        ([d_h, d], rows i d_h .. of W_V),
 * one system of size d per kept head; rho_i = rho * trace / d of that head's Gram matrix when rho_relative.
 * Reads m->X, st->P, st->Aattn (the weights in m are not read).  head_mask_host: HOST array of n_heads bytes
 * (0 = pruned; NULL = all heads kept) — the host decides which systems to build.  Wv_out: device, fp32 [d, ldw >= d],
 * rows of pruned heads are written as zero; it may be m->Wv.ptr.
 * bf16 mode: P, Aattn and the regressors are carried as bf16 hi + lo parts (the systems of the heads are worse
 * conditioned than G_X: their regressors are running averages of the inputs); fp32 mode: fp64 accumulation and
 * factorisation.
 * Workspace: sp_mha_value_refit_workspace_bytes (it holds n_heads Gram matrices of d x d floats).
 * Errors: as sp_mha_step; SP_ERR_INVALID_ARG also for rho < 0 or Wv_out == NULL; SP_ERR_NOT_SPD through status_dev.
 */
sp_status sp_mha_value_refit(const sp_mha_module* m, const sp_mha_state* st, const uint8_t* head_mask_host, double rho,
                             int32_t rho_relative, int64_t seq_chunk, float* Wv_out, int64_t ldw, int32_t* status_dev,
                             void* ws, size_t ws_bytes, void* stream);
size_t sp_mha_value_refit_workspace_bytes(int64_t d, int64_t n_heads, int64_t T, int64_t n_seq, int64_t seq_chunk,
                                          int32_t dtype);

/* ---------------------------------------------------------------------------------------------------------------
 * Helpers.
 * sp_ridge_solve   — W[m,n] = R[m,n] (G[n,n] + rho_eff I)^-1 by Cholesky and two triangular solves (weight
 *                    recovery of Appendix A.1).  G, R, W fp32; factorisation in fp64 when precise != 0, else fp32.
 *                    rho_eff as in sp_admm_params.  G is read from its lower triangle and left unchanged.
 * sp_linear_refit  — recovery on a kept support of column groups: W[:, S] = R[:, S](G[S,S] + rho_eff I)^-1,
 *                    other columns zero (Algorithm 2, "importance + recovery solver"; used for W2 and for W_O heads).
 *                    mask: u8 [n_units] with exactly k_keep ones (k_keep is a host value).  The ridge is that of the
 *                    FULL system: rho_eff = rho * trace(G)/dim(G) when rho_relative != 0 (computed on the device),
 *                    else rho.
 * sp_gemm          — C[M,N] = alpha * opA(A) opB(B) + beta * C, opX(X) = X or X^T; test and utility entry.
 *                    use_tensor_cores != 0 requests the tcgen05 path (bf16 operands only; falls back with
 *                    SP_ERR_UNSUPPORTED when shapes or alignment do not allow it).
 * sp_symmetrize    — mirror the lower triangle of a square fp32 matrix onto its upper triangle.
 */
sp_status sp_ridge_solve(const float* R, int64_t ldr, const float* G, int64_t ldg, int64_t m, int64_t n, double rho,
                         int32_t rho_relative, int32_t precise, float* W, int64_t ldw, int32_t* status_dev, void* ws,
                         size_t ws_bytes, void* stream);
sp_status sp_linear_refit(const float* R, int64_t ldr, const float* G, int64_t ldg, int64_t m, int64_t n_units,
                          int32_t group, const uint8_t* mask, int64_t k_keep, double rho, int32_t rho_relative,
                          int32_t precise, float* W, int64_t ldw, int32_t* status_dev, void* ws, size_t ws_bytes,
                          void* stream);
sp_status sp_gemm(int32_t transA, int32_t transB, int64_t M, int64_t N, int64_t K, double alpha, const sp_mat* A,
                  const sp_mat* B, double beta, const sp_mat* C, int32_t lower_only, int32_t use_tensor_cores,
                  int32_t* status_dev, void* stream);
sp_status sp_symmetrize(float* G, int64_t n, int64_t ldg, void* stream);

/* sp_set_wait_budget(cycles): every barrier wait inside the tensor-core GEMM kernel is bounded by a clock budget
 * (about two seconds by default); a wait that outlasts it makes the kernel record SP_ERR_TIMEOUT in status_dev, drain
 * its copies and tensor-core work in flight, free its tensor memory and return, leaving C incomplete.  This call
 * changes the budget process-wide (0 restores the default).  It exists for diagnosis and for testing the time-out
 * path: with a budget of a few cycles an ordinary wait for a long K loop already runs out. */
sp_status sp_set_wait_budget(int64_t cycles);

/* sp_set_reproducible(on): see "Reproducibility" at the top of this file; sp_get_reproducible() returns the setting. */
sp_status sp_set_reproducible(int32_t on);
int32_t sp_get_reproducible(void);

/* ---------------------------------------------------------------------------------------------------------------
 * Launch accounting and profiling (the paper has no counterpart; used by the benchmark).
 * sp_profile_begin(enable): resets the launch counter and the event records; enable = 1 brackets every kernel (or
 *   phase: a phase absorbs the kernels launched inside it) the library launches afterwards with a CUDA event pair on
 *   the launching stream; enable = 2 also records the kernels inside a phase (they are then counted twice).
 * sp_profile_read(out_host): after the caller synchronised the stream(s): out_host[kind*4 + {0,1,2,3}] =
 *   {records, total milliseconds, algorithmic flops, algorithmic bytes} for kind in [0, sp_profile_kinds()).
 * sp_launch_count(): kernels launched by the library since the last sp_profile_begin.
 */
sp_status sp_profile_begin(int32_t enable);
sp_status sp_profile_read(double* out_host);
int32_t sp_profile_kinds(void);
const char* sp_profile_kind_name(int32_t kind);
int64_t sp_launch_count(void);

/* Bytes of workspace the named call needs.  Meaning of (d, n, N, token_chunk, dtype) per op:
 *   SP_WS_GRAM: d = channels C, N = tokens T.   SP_WS_ADMM_STEP / SP_WS_FFN_INIT: module sizes, dtype of X.
 *   SP_WS_SCORES: d = n_units*group, N = tokens (LEMMA1) or rows of W (WANDA).
 *   SP_WS_RIDGE_SOLVE / SP_WS_LINEAR_REFIT: d = m (rows of R), n = system size, dtype SP_F64 when precise != 0.
 *   SP_WS_WEIGHT_STATS: d = number of blocks.   SP_WS_INPUT_INVERSE: d = d_model. */
size_t sp_workspace_bytes(int32_t op, int64_t d, int64_t n, int64_t N, int64_t token_chunk, int32_t dtype);
/* Optional extra workspace of sp_admm_step (bf16 mode): when ws_bytes >= sp_workspace_bytes(SP_WS_ADMM_STEP, ...) +
 * sp_admm_overlap_bytes(N, k_keep), the step keeps z^(1) = W1 X of all N tokens on the kept channels (fp32) in the
 * tail of the workspace and computes it concurrently with the recovery of W2 on the kept support; results are the
 * same, the step is faster. */
size_t sp_admm_overlap_bytes(int64_t N, int64_t k_keep);
const char* sp_status_string(int32_t status);
int32_t sp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SP_H_ */
