// bf16 tensor-core GEMM for sm_100a: TMA-fed shared-memory pipeline, tcgen05.mma with fp32 accumulators in tensor
// memory, warp-specialised persistent CTAs working in pairs.
//
//   C[M,N] = alpha * A B^T-like contraction over K + beta * Cin
//
// Both operands may be K-major (stored [rows, K], K contiguous: the weight/activation products z^(1) = X W1^T, ...)
// or MN-major (stored [K, rows], rows contiguous: the token-axis contractions A^T A, Z^T X, Ypre^T A).  Each
// major-ness has its own TMA box shape and shared-memory matrix descriptor; the MMA instruction descriptor carries
// the two major bits.
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 output tile: every CTA loads its own 128 rows of
// A and ONE HALF (128 columns) of B per k-block, and the pair's leader issues one cta_group::2 MMA of shape
// 256 x 256 x 16 that reads both halves.  A CTA therefore moves 32 KB per k-block through the L2 -> SM path instead
// of the 48 KB a lone 128 x 256 tile needs, which is what bounded the single-CTA form of this kernel.  Every load is
// an ordinary one-destination TMA load: it lands in the issuing CTA's own shared memory and completes on the
// leader's barrier.
//
// Roles (192 threads per CTA): warp 0 = TMA producer (one lane), warp 1 = tensor-memory allocator and, in the
// leader, MMA issuer (one lane), warps 2..5 = epilogue (each owns the 32 accumulator lanes its warp id maps to).  Two
// 256-column accumulators are ping-ponged so that the epilogue of tile i overlaps the main loop of tile i+1.
// Epilogue: the accumulator block of a warp (32 rows x 32 columns) goes through a 128-byte-swizzled shared tile and
// leaves by a TMA store, or a TMA add-reduction when the call accumulates into C; other cases (bf16 output, a
// separate Cin, unaligned C) use plain coalesced loads and stores through a padded tile.
// Every wait is bounded by a clock budget; on expiry the CTA records SP_ERR_TIMEOUT and leaves its loops, and both
// CTAs still meet at the final cluster barrier before tensor memory is freed.
#include <cuda.h>
#include <math.h>
#include <string.h>

#include "sp_common.cuh"

namespace sp {
namespace {

constexpr int BM = 128;            // rows of A (and of the accumulator) per CTA
constexpr int BNH = 128;           // columns of B loaded per CTA (half of the pair's tile)
constexpr int TILE_M = 2 * BM;     // tile of the CTA pair
constexpr int TILE_N = 2 * BNH;
constexpr int BK = 64;
constexpr int STAGES = 6;
constexpr int UMMA_K = 16;
constexpr int kBandRows = 8;        // tile rows per band of a lower-triangle product
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BNH * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;          // 32 KB
constexpr int STG_BYTES = 8192;                          // per epilogue warp: two 32 x 32 fp32 blocks
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 4 * STG_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr long long WAIT_BUDGET_CYCLES = 4000000000LL;   // ~2 s
constexpr long long DRAIN_BUDGET_CYCLES = 200000000LL;   // ~0.1 s

enum EpiMode : int { EPI_DIRECT = 0, EPI_TMA_STORE = 1, EPI_TMA_ADD = 2, EPI_TMA_BF16_CIN = 3 };

struct TcParams {
  int64_t M, N, K;
  float alpha, beta;
  const void* cin;
  int32_t cin_dtype;
  int64_t cin_ld;
  void* c;
  int32_t c_dtype;
  int64_t c_ld;
  int64_t c_lo_off;  // bf16 C, plain epilogue: second (lo) part of every value c_lo_off columns to the right
  int32_t a_kmajor, b_kmajor, lower_only;
  int32_t epi_mode;  // EpiMode
  int32_t n_fast;    // tile order: 1 = consecutive tiles walk N first (they share the A row block)
  TcSegments seg;    // K segments: segment s reads A at (k + a_k[s], m + a_mn[s]) and B at (k + b_k[s], n + b_mn[s])
  int32_t seg_kb;    // k-blocks per segment
  int32_t tiles_m, tiles_n, num_tiles;
  // Work units: the first n_plain tiles are one unit each (all of K).  The other n_cut = num_tiles - n_plain tiles are
  // cut along K: unit n_plain + v is tile n_plain + v % n_cut restricted to k-blocks [ks * kb_per_split,
  // (ks + 1) * kb_per_split) with ks = v / n_cut.  ksplit > 1 only with the add-reduction epilogue (partial products
  // add up in C).  n_plain = 0 cuts every tile; n_plain = whole waves of CTA pairs cuts only the tiles of the last,
  // partly filled wave, so that it keeps every pair busy for 1 / ksplit of a tile time.
  int32_t ksplit, kb_per_split, num_units, n_plain;
  // batched launches: product (b0, b1) of nb0 x nb1; tile index = product * tiles_per_batch + local tile.  The tensor
  // maps then have five dimensions; x_ord[r] is the coordinate slot (1..4) of role r = outer dimension, b0, b1, plane
  // in the map of operand x (the maps order their dimensions by stride).
  int32_t batched, nb0, nb1, tiles_per_batch;
  int8_t a_ord[4], b_ord[4], c_ord[4];
  int64_t c_s0, c_s1, cin_s0, cin_s1;
  long long wait_budget;   // clock cycles a role may wait on one barrier before it gives up (SP_ERR_TIMEOUT)
  int32_t* status;
  const int32_t* skip;     // conditional launch: every CTA returns at once when *skip != 0 (see SkipScope)
};

struct Coord5 {
  int32_t x[5];
};
__device__ __forceinline__ Coord5 make_coord(const int8_t* ord, int32_t inner, int32_t outer, int32_t b0, int32_t b1,
                                             int32_t plane) {
  Coord5 c;
  c.x[0] = inner;
  c.x[ord[0]] = outer;
  c.x[ord[1]] = b0;
  c.x[ord[2]] = b1;
  c.x[ord[3]] = plane;
  return c;
}

__device__ __forceinline__ void unit_map(const TcParams& p, int u, int num_kb, int& tile, int& kb0, int& kb1) {
  if (u < p.n_plain) {
    tile = u; kb0 = 0; kb1 = num_kb;
    return;
  }
  const int v = u - p.n_plain, n_cut = p.num_tiles - p.n_plain;
  tile = p.n_plain + v % n_cut;
  kb0 = (v / n_cut) * p.kb_per_split;
  kb1 = (kb0 + p.kb_per_split < num_kb) ? kb0 + p.kb_per_split : num_kb;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// arrive on a barrier given by its shared::cluster address (own CTA or the peer)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the budget ran out or another role of this CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget) {
  if (mbar_try(bar, parity)) return true;
  // (a try_wait may itself suspend the thread for a while, so the clock is read after every unsuccessful try)
  const long long t0 = clock64();
  while (!mbar_try(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}

// Load of one box into this CTA's shared memory; the bytes complete on the barrier `bar_cluster_addr`, which is the
// pair leader's (cta_group::2 form: the barrier may live in the peer CTA).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                            uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
      : "memory");
}
// plain one-CTA load (epilogue: a block of Cin into this warp's shared tile, completing on this CTA's barrier)
__device__ __forceinline__ void tma_load_2d_local(uint32_t dst, const CUtensorMap* map, int32_t c0, int32_t c1,
                                                  uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int32_t c0, int32_t c1, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
// five-dimensional forms for batched launches
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, const Coord5& c,
                                            uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(map), "r"(c.x[0]), "r"(c.x[1]), "r"(c.x[2]), "r"(c.x[3]), "r"(c.x[4]), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void tma_store_5d(const CUtensorMap* map, const Coord5& c, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4, %5}], [%6];"
               ::"l"(map), "r"(c.x[0]), "r"(c.x[1]), "r"(c.x[2]), "r"(c.x[3]), "r"(c.x[4]), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_5d(const CUtensorMap* map, const Coord5& c, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.5d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3, %4, %5}], [%6];"
               ::"l"(map), "r"(c.x[0]), "r"(c.x[1]), "r"(c.x[2]), "r"(c.x[3]), "r"(c.x[4]), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The MMAs issued so far by this thread arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(mask)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a 128-byte-swizzled operand tile.
//   K-major : rows of 64 bf16 (128 B); 8-row groups 1024 B apart (stride byte offset); leading offset unused (1).
//   MN-major: 64-element (128 B) runs along MN, one per K index; 8-K-index groups 1024 B apart (stride offset);
//             consecutive 64-element MN blocks `mn_block_bytes` apart (leading offset).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, bool kmajor, uint32_t mn_block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  const uint32_t lbo = kmajor ? 1u : (mn_block_bytes >> 4);
  d |= (uint64_t)(lbo & 0x3fffu) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;  // 128-byte swizzle
  return d;
}

// Instruction descriptor of the pair's MMA: 256 x 256 x 16, bf16 operands, fp32 accumulator.
__device__ __forceinline__ uint32_t make_instr_desc(bool a_kmajor, bool b_kmajor) {
  uint32_t d = 0;
  d |= 1u << 4;                          // accumulator format: fp32
  d |= 1u << 7;                          // A format: bf16
  d |= 1u << 10;                         // B format: bf16
  d |= (a_kmajor ? 0u : 1u) << 15;       // A major-ness
  d |= (b_kmajor ? 0u : 1u) << 16;       // B major-ness
  d |= (uint32_t)(TILE_N >> 3) << 17;    // N
  d |= (uint32_t)(TILE_M >> 4) << 24;    // M
  return d;
}

template <bool BATCHED>
__device__ __forceinline__ void tile_coords(const TcParams& p, int t, int& tm, int& tn, int& b0, int& b1) {
  b0 = 0;
  b1 = 0;
  if constexpr (BATCHED) {
    const int bi = t / p.tiles_per_batch;
    t -= bi * p.tiles_per_batch;
    b0 = bi % p.nb0;
    b1 = bi / p.nb0;
  }
  if (!p.lower_only) {
    if (p.n_fast) {
      tn = t % p.tiles_n;
      tm = t / p.tiles_n;
    } else {
      tm = t % p.tiles_m;
      tn = t / p.tiles_m;
    }
  } else {
    // Tiles (tm, tn) with tn <= tm of a tiles_m x tiles_n grid (tiles_m >= tiles_n: the lower triangle of a square
    // product, with any rows below the square taking part in full), walked in bands of kBandRows tile rows, column by
    // column inside a band: the tiles that run at the same time then share the band's few row panels (which stay in
    // L2) and stream each column panel once per band.
    int r0 = 0, r1 = 0;
    for (;;) {
      r1 = (r0 + kBandRows < p.tiles_m) ? r0 + kBandRows : p.tiles_m;
      int cnt = 0;
      for (int r = r0; r < r1; ++r) cnt += (r + 1 < p.tiles_n) ? r + 1 : p.tiles_n;
      if (t < cnt || r1 >= p.tiles_m) break;     // the second test only bounds the loop
      t -= cnt;
      r0 = r1;
    }
    for (tn = 0;; ++tn) {
      const int first = tn > r0 ? tn : r0;
      const int c = r1 > first ? r1 - first : 0;
      if (t < c || tn >= p.tiles_n - 1) { tm = first + (t < c ? t : 0); break; }
      t -= c;
    }
  }
}

__device__ __forceinline__ void tc_commit_local(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// BATCHED = false is the plain two-dimensional form (the products of the FFN path); BATCHED = true adds the batch
// and plane coordinates (five-dimensional tensor maps).  Two instantiations, so that the plain form carries none of
// the batched form's instructions.
template <bool BATCHED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmCin, const TcParams p) {
  if (p.skip != nullptr && *p.skip != 0) return;   // the same answer in every CTA: nothing is allocated yet
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  // identical offsets in both CTAs of the pair: the leader's MMA reads the peer's operand tiles at the offsets of
  // its own, and barrier addresses are exchanged by offset
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;            // 1024-byte aligned operand stages
  const uint32_t stg_base = tiles + STAGES * STAGE_BYTES;   // 1024-byte aligned epilogue tiles
  const uint32_t bars = stg_base + 4 * STG_BYTES;           // 8-byte aligned barrier block
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);
  auto cin_bar = [&](int q, int b) { return bars + 8u * (2 * STAGES + 5 + 2 * q + b); };   // per epilogue warp

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
  const int cid = (int)(blockIdx.x >> 1);        // pair index
  const int ncl = (int)(gridDim.x >> 1);
  volatile int* abort_flag = &s_abort;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }   // 4 warps x 2 CTAs
    mbar_init(drain_bar, 1);
    for (int q = 0; q < 4; ++q) { mbar_init(cin_bar(q, 0), 1); mbar_init(cin_bar(q, 1), 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {   // the same warp in both CTAs allocates the pair's tensor memory
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();      // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;

  const int num_kb = p.seg_kb * p.seg.nseg;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int u = cid; u < p.num_units && ok; u += ncl) {
        int tm, tn, tile, kb0, kb1, b0, b1;
        unit_map(p, u, num_kb, tile, kb0, kb1);
        tile_coords<BATCHED>(p, tile, tm, tn, b0, b1);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.wait_budget)) { ok = false; break; }
          // the leader's barrier collects the bytes of both CTAs' loads of this stage
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
          const uint32_t fbar = map_to_cta(full_bar(s), 0);
          const uint32_t a_dst = tiles + s * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const int sg = kb / p.seg_kb;
          const int kk = (kb - sg * p.seg_kb) * BK;
          const int ka = kk + p.seg.a_k[sg], kbb = kk + p.seg.b_k[sg];
          const int am = tm * TILE_M + (int)rank * BM + p.seg.a_mn[sg];
          const int bn = tn * TILE_N + (int)rank * BNH + p.seg.b_mn[sg];
          if constexpr (BATCHED) {
            const int pa = p.seg.a_p[sg], pb = p.seg.b_p[sg];
            if (p.a_kmajor) {
              tma_load_5d(a_dst, &tmA, make_coord(p.a_ord, ka, am, b0, b1, pa), fbar);
            } else {
#pragma unroll
              for (int mb = 0; mb < BM / 64; ++mb)
                tma_load_5d(a_dst + mb * (64 * BK * 2), &tmA, make_coord(p.a_ord, am + mb * 64, ka, b0, b1, pa), fbar);
            }
            if (p.b_kmajor) {
              tma_load_5d(b_dst, &tmB, make_coord(p.b_ord, kbb, bn, b0, b1, pb), fbar);
            } else {
#pragma unroll
              for (int nb = 0; nb < BNH / 64; ++nb)
                tma_load_5d(b_dst + nb * (64 * BK * 2), &tmB, make_coord(p.b_ord, bn + nb * 64, kbb, b0, b1, pb), fbar);
            }
          } else {
            if (p.a_kmajor) {
              tma_load_2d(a_dst, &tmA, ka, am, fbar);
            } else {
#pragma unroll
              for (int mb = 0; mb < BM / 64; ++mb) tma_load_2d(a_dst + mb * (64 * BK * 2), &tmA, am + mb * 64, ka, fbar);
            }
            if (p.b_kmajor) {
              tma_load_2d(b_dst, &tmB, kbb, bn, fbar);
            } else {
#pragma unroll
              for (int nb = 0; nb < BNH / 64; ++nb) tma_load_2d(b_dst + nb * (64 * BK * 2), &tmB, bn + nb * 64, kbb, fbar);
            }
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        report_status(p.status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 1);
        // give copies already in flight time to land before shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < DRAIN_BUDGET_CYCLES) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_instr_desc(p.a_kmajor != 0, p.b_kmajor != 0);
      int s = 0;
      uint32_t ph = 0;
      int acc = 0;
      uint32_t aph = 0;
      bool ok = true;
      bool issued = false;
      for (int u = cid; u < p.num_units && ok; u += ncl) {
        if (!mbar_wait(tempty_bar(acc), aph ^ 1u, abort_flag, p.wait_budget)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TILE_N);
        int tile, kb0, kb1;
        unit_map(p, u, num_kb, tile, kb0, kb1);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(s), ph, abort_flag, p.wait_budget)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles + s * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // K-major: 16 bf16 = 32 B further along the swizzled row; MN-major: 16 K indices = 16 * 128 B further
            const uint32_t a_off = p.a_kmajor ? (uint32_t)(k * UMMA_K * 2) : (uint32_t)(k * UMMA_K * 128);
            const uint32_t b_off = p.b_kmajor ? (uint32_t)(k * UMMA_K * 2) : (uint32_t)(k * UMMA_K * 128);
            const uint64_t adesc = make_smem_desc(a_src + a_off, p.a_kmajor != 0, 64 * BK * 2);
            const uint64_t bdesc = make_smem_desc(b_src + b_off, p.b_kmajor != 0, 64 * BK * 2);
            tc_mma_bf16_pair(d_tmem, adesc, bdesc, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          issued = true;
          tc_commit_pair(empty_bar(s));   // frees the stage in both CTAs once these MMAs have read it
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar(acc));   // accumulator complete: wakes the epilogue warps of both CTAs
        if (++acc == 2) { acc = 0; aph ^= 1u; }
      }
      if (!ok) report_status(p.status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 2);
      // Wait for the MMAs in flight before shared and tensor memory are released.  In a complete run the epilogue
      // has already seen the last accumulator, so this returns at once; it matters when a role gave up (here, or an
      // epilogue warp that left without waiting for its accumulator).
      if (issued && (!ok || *abort_flag)) {
        tc_commit_local(drain_bar);
        const long long t0 = clock64();
        while (!mbar_try(drain_bar, 0u) && clock64() - t0 < DRAIN_BUDGET_CYCLES) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 2..5 (both CTAs)
    // tcgen05.ld hands every lane one accumulator row (32 consecutive columns per load).
    const int q = warp & 3;                 // accumulator lane quarter this warp may read
    const uint32_t wstg = stg_base + (uint32_t)q * STG_BYTES;
    uint8_t* wstg_ptr = smem_raw + (wstg - raw);
    float (*stg)[33] = reinterpret_cast<float (*)[33]>(wstg_ptr);   // padded tile of the plain path
    const uint32_t tempty_leader[2] = {map_to_cta(tempty_bar(0), 0), map_to_cta(tempty_bar(1), 0)};
    int acc = 0;
    uint32_t aph = 0;
    int buf = 0, cbuf = 0;
    uint32_t cph = 0;           // phase bit of each of the two Cin barriers
    bool ok = true;
    const bool has_cin = p.beta != 0.f;
    const bool cin_f32 = p.cin_dtype == SP_F32, c_f32 = p.c_dtype == SP_F32;
    for (int u = cid; u < p.num_units && ok; u += ncl) {
      int tm, tn, tile, kb0_unused, kb1_unused, b0, b1;
      unit_map(p, u, num_kb, tile, kb0_unused, kb1_unused);
      tile_coords<BATCHED>(p, tile, tm, tn, b0, b1);
      const int64_t c_boff = BATCHED ? (int64_t)b0 * p.c_s0 + (int64_t)b1 * p.c_s1 : 0;
      const int64_t cin_boff = BATCHED ? (int64_t)b0 * p.cin_s0 + (int64_t)b1 * p.cin_s1 : 0;
      // every lane observes the barrier itself; the vote keeps the warp converged for the aligned TMEM loads
      const bool got = mbar_wait(tfull_bar(acc), aph, abort_flag, p.wait_budget);
      if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
      tc_fence_after();
      const int64_t row0 = (int64_t)tm * TILE_M + (int64_t)rank * BM + q * 32;   // first global row of this warp
      const uint32_t taddr = tmem_base + (uint32_t)(acc * TILE_N) + ((uint32_t)(q * 32) << 16);
      const int rows_here = (p.M - row0 < 32) ? (int)(p.M - row0) : 32;   // may be <= 0 on a ragged last tile
      if (p.epi_mode == EPI_TMA_BF16_CIN) {
        // bf16 C = beta * Cin + alpha * acc with both matrices moved by TMA: the warp's tile holds two 32 x 32 bf16
        // blocks of Cin (loaded one block ahead) and two blocks of C.  64-byte rows, 64-byte swizzle: 16-byte chunk j
        // of row r sits at chunk j ^ ((r >> 1) & 3).
        const bool rows_ok = rows_here > 0;
        const int nsl = (int)(((p.N - (int64_t)tn * TILE_N < TILE_N) ? (p.N - (int64_t)tn * TILE_N) : TILE_N) + 31) / 32;
        if (rows_ok && lane == 0 && nsl > 0) {
          fence_async_smem();
          mbar_expect_tx(cin_bar(q, cbuf), 2048);
          tma_load_2d_local(wstg + cbuf * 2048, &tmCin, (int32_t)((int64_t)tn * TILE_N), (int32_t)row0, cin_bar(q, cbuf));
        }
#pragma unroll 1
        for (int sl = 0; sl < nsl; ++sl) {
          const int64_t gj0 = (int64_t)tn * TILE_N + sl * 32;
          uint32_t r[32];
          tc_ld32(taddr + (uint32_t)(sl * 32), r);
          tc_wait_ld();
          if (rows_ok) {
            if (lane == 0 && sl + 1 < nsl) {     // next block of Cin into the other half (its last reader is done)
              fence_async_smem();
              mbar_expect_tx(cin_bar(q, cbuf ^ 1), 2048);
              tma_load_2d_local(wstg + (cbuf ^ 1) * 2048, &tmCin, (int32_t)(gj0 + 32), (int32_t)row0,
                                cin_bar(q, cbuf ^ 1));
            }
            const bool got_c = mbar_wait(cin_bar(q, cbuf), (cph >> cbuf) & 1u, abort_flag, p.wait_budget);
            if (!__all_sync(0xffffffffu, got_c)) { ok = false; break; }
            if (lane == 0) bulk_wait_read_1();
            __syncwarp();
            const uint8_t* in_row = wstg_ptr + cbuf * 2048 + lane * 64;
            uint8_t* out_row = wstg_ptr + 4096 + buf * 2048 + lane * 64;
            const int sw = (lane >> 1) & 3;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 cw = *reinterpret_cast<const uint4*>(in_row + ((j ^ sw) << 4));
              const uint32_t cwv[4] = {cw.x, cw.y, cw.z, cw.w};
              uint32_t ow[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 c2 = *reinterpret_cast<const __nv_bfloat162*>(&cwv[e]);
                const float v0 = fmaf(p.beta, __low2float(c2), p.alpha * __uint_as_float(r[8 * j + 2 * e]));
                const float v1 = fmaf(p.beta, __high2float(c2), p.alpha * __uint_as_float(r[8 * j + 2 * e + 1]));
                const __nv_bfloat162 o2 = __floats2bfloat162_rn(v0, v1);
                ow[e] = *reinterpret_cast<const uint32_t*>(&o2);
              }
              *reinterpret_cast<uint4*>(out_row + ((j ^ sw) << 4)) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmC, (int32_t)gj0, (int32_t)row0, wstg + 4096 + buf * 2048);
              bulk_commit();
            }
            cph ^= 1u << cbuf;
            cbuf ^= 1;
            buf ^= 1;
          }
        }
        if (!ok) break;
      } else if (p.epi_mode != EPI_DIRECT) {
        // 32 x 32 fp32 block -> 128-byte-swizzled shared tile (16-byte chunk j of row r sits at chunk j ^ (r & 7))
        // -> one TMA store / add-reduction, which clips at the edges of C.  Two tiles per warp alternate.
#pragma unroll 1
        for (int c0 = 0; c0 < TILE_N; c0 += 32) {
          const int64_t gj0 = (int64_t)tn * TILE_N + c0;
          if (gj0 >= p.N) break;                  // uniform over the warp
          uint32_t r[32];
          tc_ld32(taddr + (uint32_t)c0, r);
          tc_wait_ld();
          if (lane == 0) bulk_wait_read_1();      // the copy that last read this tile (two blocks ago) is done
          __syncwarp();
          uint8_t* tile = wstg_ptr + buf * 4096 + lane * 128;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float4 v = make_float4(p.alpha * __uint_as_float(r[4 * j]), p.alpha * __uint_as_float(r[4 * j + 1]),
                                         p.alpha * __uint_as_float(r[4 * j + 2]), p.alpha * __uint_as_float(r[4 * j + 3]));
            *reinterpret_cast<float4*>(tile + ((j ^ (lane & 7)) << 4)) = v;
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (rows_here > 0) {
              if constexpr (BATCHED) {
                const Coord5 cc = make_coord(p.c_ord, (int32_t)gj0, (int32_t)row0, b0, b1, 0);
                if (p.epi_mode == EPI_TMA_STORE) tma_store_5d(&tmC, cc, wstg + buf * 4096);
                else tma_reduce_add_5d(&tmC, cc, wstg + buf * 4096);
              } else {
                if (p.epi_mode == EPI_TMA_STORE) tma_store_2d(&tmC, (int32_t)gj0, (int32_t)row0, wstg + buf * 4096);
                else tma_reduce_add_2d(&tmC, (int32_t)gj0, (int32_t)row0, wstg + buf * 4096);
              }
            }
            bulk_commit();
          }
          buf ^= 1;
        }
      } else {
        // plain path: the block is turned through a padded tile so that global loads and stores see a warp on 32
        // consecutive columns of one row (128-byte lines) instead of 32 different rows
#pragma unroll 1
        for (int c0 = 0; c0 < TILE_N; c0 += 32) {
          const int64_t gj0 = (int64_t)tn * TILE_N + c0;
          if (gj0 >= p.N) break;                  // uniform over the warp
          const int64_t gj = gj0 + lane;
          // the 32 rows of Cin for this column are fetched first (independent loads in flight while the accumulator
          // block is read from tensor memory and turned)
          float cv[32];
          if (has_cin) {
            const int64_t cin_off = cin_boff + row0 * p.cin_ld + gj;
#pragma unroll
            for (int rr = 0; rr < 32; ++rr) {
              cv[rr] = 0.f;
              if (gj < p.N && rr < rows_here) {
                const int64_t o = cin_off + (int64_t)rr * p.cin_ld;
                cv[rr] = cin_f32 ? reinterpret_cast<const float*>(p.cin)[o]
                                 : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.cin)[o]);
              }
            }
          }
          uint32_t r[32];
          tc_ld32(taddr + (uint32_t)c0, r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) stg[lane][i] = p.alpha * __uint_as_float(r[i]);
          __syncwarp();
          if (gj < p.N) {
            const int64_t c_off = c_boff + row0 * p.c_ld + gj;
#pragma unroll
            for (int rr = 0; rr < 32; ++rr) {
              if (rr < rows_here) {
                float v = stg[rr][lane];
                if (has_cin) v = fmaf(p.beta, cv[rr], v);
                const int64_t o = c_off + (int64_t)rr * p.c_ld;
                if (c_f32) {
                  reinterpret_cast<float*>(p.c)[o] = v;
                } else {
                  const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                  reinterpret_cast<__nv_bfloat16*>(p.c)[o] = hi;
                  if (p.c_lo_off > 0)
                    reinterpret_cast<__nv_bfloat16*>(p.c)[o + p.c_lo_off] = __float2bfloat16_rn(v - __bfloat162float(hi));
                }
              }
            }
          }
          __syncwarp();
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_leader[acc]);   // the leader's MMA thread counts both CTAs' warps
      if (++acc == 2) { acc = 0; aph ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();         // shared tiles and C are settled before the CTA leaves
    if (!ok && lane == 0) report_status(p.status, SP_ERR_TIMEOUT, (int32_t)blockIdx.x, 3);
  }

  // both CTAs are done with each other's shared memory and barriers before either leaves
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Tensor map of a row-major matrix [outer, inner] with leading dimension ld (elements), 128-byte swizzle.
//   bf16 operand, K-major : inner = K, outer = rows, box = {64, 128}
//   bf16 operand, MN-major: inner = rows, outer = K, box = {64, 64}
//   fp32 output C         : inner = N, outer = M, box = {32, 32}
//   bf16 C / Cin          : inner = N, outer = M, box = {32, 32}, 64-byte swizzle
bool make_map(CUtensorMap* map, bool f32, const void* ptr, int64_t inner, int64_t outer, int64_t ld, int box_inner,
              int box_outer, bool swizzle64 = false) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                  const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

namespace {
// Five-dimensional tensor map of a batched operand.  Roles: inner (contiguous) dimension, outer dimension (stride ld),
// batch dimensions b0 and b1, plane.  The non-inner dimensions are laid out in the map by ascending stride (extent-1
// dimensions last); ord[r] receives the slot (1..4) of role r = outer, b0, b1, plane.  Boxes are 1 deep in b0, b1, plane.
bool make_map5(CUtensorMap* map, bool f32, const void* ptr, int64_t inner, int box_inner, int64_t outer, int64_t ld,
               int box_outer, int64_t nb0, int64_t s0, int64_t nb1, int64_t s1, int64_t planes, int64_t plane_stride,
               bool swizzle_none_ok, int8_t ord[4]) {
  (void)swizzle_none_ok;
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const int64_t es = f32 ? 4 : 2;
  struct Dim { int64_t ext, stride; int box, role; };
  Dim dm[4] = {{outer, ld, box_outer, 0}, {nb0, s0, 1, 1}, {nb1, s1, 1, 2}, {planes, plane_stride, 1, 3}};
  // insertion sort by (extent == 1, stride)
  for (int i = 1; i < 4; ++i)
    for (int j = i; j > 0; --j) {
      const bool a1 = dm[j - 1].ext <= 1, b1 = dm[j].ext <= 1;
      const bool swap = (a1 && !b1) || (a1 == b1 && !a1 && dm[j].stride < dm[j - 1].stride);
      if (!swap) break;
      const Dim t = dm[j - 1]; dm[j - 1] = dm[j]; dm[j] = t;
    }
  cuuint64_t dims[5] = {(cuuint64_t)inner, 1, 1, 1, 1};
  cuuint64_t strides[4];
  cuuint32_t box[5] = {(cuuint32_t)box_inner, 1, 1, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  int64_t last = 16;
  for (int i = 0; i < 4; ++i) {
    dims[i + 1] = (cuuint64_t)(dm[i].ext > 0 ? dm[i].ext : 1);
    box[i + 1] = (cuuint32_t)dm[i].box;
    int64_t st = dm[i].stride * es;
    if (dm[i].ext <= 1 && dm[i].role != 0) st = last;     // unused dimension: any legal stride
    if (st <= 0 || st % 16 != 0) return false;
    strides[i] = (cuuint64_t)st;
    last = st > last ? st : last;
    ord[dm[i].role] = (int8_t)(i + 1);
  }
  CUresult r = fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5,
                  const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}
}  // namespace

int sm_count() {
  static std::mutex mu;
  static int table[PerDeviceOnce::kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return 148;
  std::lock_guard<std::mutex> guard(mu);
  if (table[dev] == 0) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    table[dev] = n > 0 ? n : 148;
  }
  return table[dev];
}

bool gemm_tc_supported(int64_t M, int64_t N, int64_t K, TcOperand A, TcOperand B) {
  if (M <= 0 || N <= 0 || K <= 0) return false;
  if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return false;
  if ((reinterpret_cast<uintptr_t>(A.ptr) & 15u) || (reinterpret_cast<uintptr_t>(B.ptr) & 15u)) return false;
  if (A.ld % 8 != 0 || B.ld % 8 != 0) return false;
  return true;
}

sp_status gemm_tc(int64_t M, int64_t N, int64_t K, float alpha, TcOperand A, TcOperand B, float beta, Operand Cin,
                  OutOperand C, bool lower_only, int32_t* status_dev, cudaStream_t stream, const TcSegments* segs,
                  double alg_flops, int max_pairs, const TcBatch* batch) {
  const bool batched = batch != nullptr;
  if (batched && (lower_only || batch->nb0 < 1 || batch->nb1 < 1 || batch->a_planes < 1 || batch->b_planes < 1))
    return SP_ERR_INVALID_ARG;
  TcSegments sg;
  if (segs) sg = *segs;
  else { sg = TcSegments{}; sg.nseg = 1; }
  if (sg.nseg < 1 || sg.nseg > kTcMaxSegments) return SP_ERR_INVALID_ARG;
  // extents of the stored operands along K and along M / N (the tensor maps zero-fill beyond them)
  const int64_t a_kext = A.kext > 0 ? A.kext : K, b_kext = B.kext > 0 ? B.kext : K;
  const int64_t a_mext = A.mnext > 0 ? A.mnext : M, b_next = B.mnext > 0 ? B.mnext : N;
  if (M <= 0 || N <= 0 || K <= 0) return SP_ERR_SHAPE;
  if (!gemm_tc_supported(M, N, K, A, B)) return SP_ERR_UNSUPPORTED;
  for (int i = 0; i < sg.nseg; ++i) {
    // TMA: the innermost coordinate times the element size must be a multiple of 16 bytes
    const int a_inner = A.kmajor ? sg.a_k[i] : sg.a_mn[i], b_inner = B.kmajor ? sg.b_k[i] : sg.b_mn[i];
    if (a_inner % 8 != 0 || b_inner % 8 != 0) return SP_ERR_ALIGNMENT;
    if (sg.a_k[i] < 0 || sg.a_mn[i] < 0 || sg.b_k[i] < 0 || sg.b_mn[i] < 0) return SP_ERR_INVALID_ARG;
  }
  if (lower_only && M < N) return SP_ERR_SHAPE;
  if (beta != 0.f && (Cin.ptr == nullptr || Cin.s1 != 1)) return SP_ERR_INVALID_ARG;
  if (C.dtype != SP_F32 && C.dtype != SP_BF16) return SP_ERR_DTYPE;
  if (beta != 0.f && Cin.dtype != SP_F32 && Cin.dtype != SP_BF16) return SP_ERR_DTYPE;

  CUtensorMap tmA, tmB, tmC, tmCin;
  memset(&tmC, 0, sizeof(tmC));
  memset(&tmCin, 0, sizeof(tmCin));
  TcParams p;
  memset(&p, 0, sizeof(p));
  bool ok;
  if (batched) {
    const TcBatch& bt = *batch;
    for (int i = 0; i < sg.nseg; ++i)
      if (sg.a_p[i] < 0 || sg.a_p[i] >= bt.a_planes || sg.b_p[i] < 0 || sg.b_p[i] >= bt.b_planes)
        return SP_ERR_INVALID_ARG;
    ok = A.kmajor ? make_map5(&tmA, false, A.ptr, a_kext, BK, a_mext, A.ld, BM, bt.nb0, bt.a_s0, bt.nb1, bt.a_s1,
                              bt.a_planes, bt.a_plane, true, p.a_ord)
                  : make_map5(&tmA, false, A.ptr, a_mext, 64, a_kext, A.ld, BK, bt.nb0, bt.a_s0, bt.nb1, bt.a_s1,
                              bt.a_planes, bt.a_plane, true, p.a_ord);
    ok = ok && (B.kmajor ? make_map5(&tmB, false, B.ptr, b_kext, BK, b_next, B.ld, BNH, bt.nb0, bt.b_s0, bt.nb1,
                                     bt.b_s1, bt.b_planes, bt.b_plane, true, p.b_ord)
                         : make_map5(&tmB, false, B.ptr, b_next, 64, b_kext, B.ld, BK, bt.nb0, bt.b_s0, bt.nb1,
                                     bt.b_s1, bt.b_planes, bt.b_plane, true, p.b_ord));
    if (!ok) return SP_ERR_ALIGNMENT;
  } else {
    ok = A.kmajor ? make_map(&tmA, false, A.ptr, a_kext, a_mext, A.ld, BK, BM)
                  : make_map(&tmA, false, A.ptr, a_mext, a_kext, A.ld, 64, BK);
    ok = ok && (B.kmajor ? make_map(&tmB, false, B.ptr, b_kext, b_next, B.ld, BK, BNH)
                         : make_map(&tmB, false, B.ptr, b_next, b_kext, B.ld, 64, BK));
    if (!ok) return SP_ERR_CUDA;
  }
  p.batched = batched ? 1 : 0;
  p.nb0 = batched ? batch->nb0 : 1;
  p.nb1 = batched ? batch->nb1 : 1;
  p.c_s0 = batched ? batch->c_s0 : 0; p.c_s1 = batched ? batch->c_s1 : 0;
  p.cin_s0 = batched ? batch->cin_s0 : 0; p.cin_s1 = batched ? batch->cin_s1 : 0;

  p.M = M; p.N = N; p.K = K;
  p.alpha = alpha; p.beta = beta;
  p.cin = Cin.ptr; p.cin_dtype = Cin.dtype; p.cin_ld = Cin.s0;
  p.c = C.ptr; p.c_dtype = C.dtype; p.c_ld = C.ld;
  p.c_lo_off = C.dtype == SP_BF16 ? C.lo_off : 0;
  if (C.lo_off < 0 || (C.lo_off > 0 && C.dtype != SP_BF16)) return SP_ERR_INVALID_ARG;
  p.a_kmajor = A.kmajor ? 1 : 0;
  p.b_kmajor = B.kmajor ? 1 : 0;
  p.lower_only = lower_only ? 1 : 0;
  // fp32 C that a tensor map can describe leaves through TMA: a store when nothing is added, an add-reduction when
  // the call accumulates into C itself (each element of C is touched once per launch, so the result is the same sum)
  p.epi_mode = EPI_DIRECT;
  // (a bulk tensor store moves whole 16-byte pieces: with N % 4 != 0 the last piece of a row would reach past
  // column N and overwrite up to three floats that belong to the caller)
  bool c_tma = C.dtype == SP_F32 && C.ld % 4 == 0 && N % 4 == 0 && (reinterpret_cast<uintptr_t>(C.ptr) & 15u) == 0;
  if (batched && ((batch->nb0 > 1 && batch->c_s0 % 4 != 0) || (batch->nb1 > 1 && batch->c_s1 % 4 != 0))) c_tma = false;
  if (c_tma && beta == 0.f) p.epi_mode = EPI_TMA_STORE;
  if (c_tma && beta == 1.f && Cin.ptr == C.ptr && Cin.dtype == SP_F32 && Cin.s0 == C.ld &&
      (!batched || (batch->cin_s0 == batch->c_s0 && batch->cin_s1 == batch->c_s1)))
    p.epi_mode = EPI_TMA_ADD;
  if (p.epi_mode != EPI_DIRECT) {
    if (batched) {
      if (!make_map5(&tmC, true, C.ptr, N, 32, M, C.ld, 32, batch->nb0, batch->c_s0, batch->nb1, batch->c_s1, 1, 0,
                     true, p.c_ord))
        return SP_ERR_CUDA;
    } else if (!make_map(&tmC, true, C.ptr, N, M, C.ld, 32, 32)) {
      return SP_ERR_CUDA;
    }
  }
  // bf16 C = beta * Cin + alpha * acc with a bf16 Cin: both through TMA
  if (p.epi_mode == EPI_DIRECT && !batched && p.c_lo_off == 0 && beta != 0.f && C.dtype == SP_BF16 && Cin.dtype == SP_BF16 &&
      C.ld % 8 == 0 && N % 8 == 0 &&
      Cin.s0 % 8 == 0 && (reinterpret_cast<uintptr_t>(C.ptr) & 15u) == 0 &&
      (reinterpret_cast<uintptr_t>(Cin.ptr) & 15u) == 0) {
    if (!make_map(&tmC, false, C.ptr, N, M, C.ld, 32, 32, true) ||
        !make_map(&tmCin, false, Cin.ptr, N, M, Cin.s0, 32, 32, true))
      return SP_ERR_CUDA;
    p.epi_mode = EPI_TMA_BF16_CIN;
  }
  p.seg = sg;
  p.seg_kb = (int32_t)ceil_div(K, BK);
  p.tiles_m = (int32_t)ceil_div(M, TILE_M);
  p.tiles_n = (int32_t)ceil_div(N, TILE_N);
  // consecutive tiles (which run at the same time on neighbouring SMs) should share the larger operand panel
  p.n_fast = p.tiles_n < p.tiles_m ? 1 : 0;
  if (lower_only) {
    int64_t cnt = 0;
    for (int tn = 0; tn < p.tiles_n && tn < p.tiles_m; ++tn) cnt += p.tiles_m - tn;
    p.num_tiles = (int32_t)cnt;
  } else {
    p.num_tiles = p.tiles_m * p.tiles_n;
  }
  p.tiles_per_batch = p.num_tiles;
  if (batched) {
    const int64_t all = (int64_t)p.num_tiles * batch->nb0 * batch->nb1;
    if (all > 0x7fffffff) return SP_ERR_SHAPE;
    p.num_tiles = (int32_t)all;
  }
  p.status = status_dev;
  p.wait_budget = wait_budget_cycles() > 0 ? wait_budget_cycles() : WAIT_BUDGET_CYCLES;
  p.skip = skip_flag();

  // Tile counts that do not fill the last wave of CTA pairs leave SMs idle.  A call that accumulates into C through
  // the add-reduction epilogue may cut K into a few ranges per tile instead: the partial products add up in C (in an
  // order that is not fixed, so the last bits of such sums can differ between runs).  A plain store into an fp32 C
  // is turned into "clear C, then accumulate" when that pays.
  int pairs_max = sm_count() / 2;
  if (max_pairs > 0 && max_pairs < pairs_max) pairs_max = max_pairs;
  const int num_kb = p.seg_kb * sg.nseg;
  p.ksplit = 1;
  const bool may_cut = !batched && !reproducible_mode();   // partial products of a cut tile add in no fixed order
  if (may_cut && (p.epi_mode == EPI_TMA_STORE || p.epi_mode == EPI_TMA_ADD) && p.num_tiles > 0) {
    auto eff = [&](int ks) {
      const double u = (double)p.num_tiles * ks;
      return u / (ceil(u / pairs_max) * pairs_max);
    };
    int best = 1;
    for (int ks = 2; ks <= 4; ++ks)
      if (num_kb / ks >= 32 && eff(ks) > eff(best) + 0.03) best = ks;
    if (best > 1 && p.epi_mode == EPI_TMA_STORE && p.skip != nullptr) best = 1;   // no unconditional clear of C
    if (best > 1) {
      if (p.epi_mode == EPI_TMA_STORE) {
        if (cudaMemset2DAsync(C.ptr, (size_t)C.ld * 4, 0, (size_t)N * 4, (size_t)M, stream) != cudaSuccess)
          return SP_ERR_CUDA;
        p.epi_mode = EPI_TMA_ADD;
      }
      p.ksplit = best;
    }
  }
  p.n_plain = 0;
  if (may_cut && p.epi_mode == EPI_TMA_ADD && p.num_tiles > pairs_max && p.num_tiles % pairs_max != 0) {
    // Alternative: whole waves of uncut tiles, and only the tiles of the last wave cut, as many ways as pairs are
    // left per tile.  Times in units of one tile on one pair.
    const int full = p.num_tiles / pairs_max, rem = p.num_tiles % pairs_max;
    int ways = pairs_max / rem;
    if (ways > 8) ways = 8;
    while (ways > 1 && num_kb / ways < 32) --ways;
    const double t_uniform = ceil((double)p.num_tiles * p.ksplit / pairs_max) / p.ksplit;
    const double t_tail = full + 1.0 / ways;
    if (ways > 1 && t_tail < 0.99 * t_uniform) {
      p.n_plain = full * pairs_max;
      p.ksplit = ways;
    }
  }
  p.kb_per_split = (int32_t)ceil_div(num_kb, p.ksplit);
  p.ksplit = (int32_t)ceil_div(num_kb, p.kb_per_split);
  p.num_units = p.n_plain + (p.num_tiles - p.n_plain) * p.ksplit;

  static PerDeviceOnce attr_once;
  if (attr_once.run([] {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)SMEM_BYTES);
        if (e == cudaSuccess)
          e = cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
        return e;
      }) != cudaSuccess)
    return SP_ERR_CUDA;
  count_launch();
  // lower-only: the triangle of the leading N x N square and all of the M - N rows below it
  const double flops = alg_flops >= 0.0 ? alg_flops
                       : lower_only     ? (double)K * (double)N * (2.0 * (double)M - (double)N)
                                        : 2.0 * (double)M * (double)N * (double)K * p.nb0 * p.nb1;
  ProfScope prof(p.skip != nullptr ? PK_CONDITIONAL : max_pairs > 0 ? PK_GEMM_TC_SHARED : PK_GEMM_TC,
                 p.skip != nullptr ? 0.0 : flops, 0.0, stream);
  const int pairs = p.num_units < pairs_max ? p.num_units : pairs_max;
  if (batched) gemm_tc_kernel<true><<<2 * pairs, NUM_THREADS, SMEM_BYTES, stream>>>(tmA, tmB, tmC, tmCin, p);
  else gemm_tc_kernel<false><<<2 * pairs, NUM_THREADS, SMEM_BYTES, stream>>>(tmA, tmB, tmC, tmCin, p);
  return cudaGetLastError() == cudaSuccess ? SP_OK : SP_ERR_CUDA;
}

}  // namespace sp
