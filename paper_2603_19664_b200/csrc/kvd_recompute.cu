// Fused K/V recomputation kernel (paper Eq. 13-14 with Eq. 1-2 and Eq. 11-12 folded in).
//
//   Y[M, 2*n_kv*d_head] = X[M, d_hidden] * W'          W' = diag(gamma) W_kv, bf16, K-major
//   (the M rows of one launch may come from several sources -- ranges of the residual store of
//    several sequences plus one caller buffer; each source owns a run of 256-row blocks)
//   y <- y / sqrt(mean_i x_i^2 + eps)                   RMSNorm applied after the contraction
//   K heads: optional RMS norm over d_head, scale gamma_k, rotation by the row's position
//   K, V stored as bf16
//
// Persistent CTA pairs (clusters of two, one CTA per SM) walk over 256 x BLOCK_N output tiles with
// tcgen05.mma.cta_group::2: each CTA owns 128 rows of the tile and stages, per 64-wide k block, its
// own 128x64 tile of X plus HALF of the BLOCK_Nx64 tile of W'; the tensor cores of the pair read
// both halves, so a k block costs each SM 32 KB of L2 traffic instead of 48 KB.  Both CTAs' loads
// count their bytes on ONE barrier per stage, in the even CTA, which that CTA's producer arms for
// the pair: the MMA issuer waits on a single barrier and nothing has to be relayed across the pair.
// Warp roles:
//   warp 2         TMA producer (one lane)
//   warp 3         even CTA: one lane issues the MMAs for the pair and commits to both CTAs' barriers;
//                  owns the TMEM allocation
//   warps 0,1,8,9  row statistics 1/rms(x): read back from the store for checkpointed rows (taken
//                  when the row was checkpointed), taken from global memory for the caller's rows
//   warps 4-7      epilogue: tcgen05.ld the fp32 accumulator, normalise, rotate, convert, store
// Nothing but the tensor cores reads the operand ring, so a stage is free again as soon as the MMAs
// that read it have retired.  Warp w runs on scheduler w % 4, so the two single-thread roles (warps
// 2, 3) share their scheduler with one epilogue warp only.
// The accumulator is double-buffered in TMEM (2 x BLOCK_N columns) so the epilogue of tile i
// overlaps the main loop of tile i+1.
//
// The producer and the MMA issuer are single threads whose loop must finish well inside the 512
// clocks a k block of MMAs takes; their loops are therefore kept to a few dozen instructions
// (incremental addresses, one asm block per k block).  Every wait is bounded; on expiry the kernel
// records STATUS_TIMEOUT and drains.
//
// Bit-reproducibility: the k loop always runs over all of d_hidden in ascending order with one MMA
// shape, a row's sum of squares is taken by one function in one fixed order wherever it is taken
// (warp_rows_sumsq), the key norm is reduced by the single thread that owns the row, and cos/sin
// depend on (position, channel) only.  A row's output bits are therefore independent of M, of the
// row's index and of whether it came from the store or from the caller.
//
// Variants of the one kernel (template arguments):
//   FG > 0  recompute fused into attention (kvd_decode_attention_recompute): for a job that carries a
//           query the key tile's epilogue turns keys into scores and the value tile is produced
//           transposed and reduced with the softmax weights; nothing of K or V is written.
//   EB = 1  FP8 checkpoints (kvd_recompute_kv_fp8): rows and weights are E4M3 codes, a k block is 128
//           channels, the MMA kind is f8f6f4; the scales ride in the per-row factor of the epilogue.
//           Combines with FG > 0 (kvd_decode_attention_recompute_fp8).
//   DT = 1  fp16 rows, weights and outputs (kvd_set_dtype), plain variant only.
#include <math_constants.h>
#include <string.h>

#include <type_traits>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

// FG = 0: the plain kernel (K and V are stored).  FG > 0: the fused variant for models with FG query
// heads per KV head -- jobs that carry a query attend over their rows inside the kernel (see the
// epilogue); it gives one ring stage to the score buffers.
// LOSM: the low rotation table (d_head/2 pairs x 16 positions, 64 B per channel) sits in shared memory
// instead of being read through L1.  The table and the high table's rows do not fit the L1 that is left
// beside the ring (a third of the epilogue's global loads miss, and a key tile's epilogue spends more
// than half its time on them); in shared memory the table costs a ring stage.  Launches whose key-tile
// epilogues are exposed (one tile per cluster; the FP8 variant, whose main loop is shorter than that
// epilogue; the fused variant, which has given a stage away already) take LOSM, the others the seventh
// stage.  The arithmetic is the same either way.
template <int BLOCK_N, int D_HEAD, int FG = 0, bool LOSM = false>
struct RcCfg {
  static constexpr bool FUSED = FG > 0;
  static_assert(!FUSED || LOSM, "the fused variant keeps the low table in shared memory");
  static constexpr int STAGES = (BLOCK_N == 256 ? 7 : 9) - ((FUSED || LOSM) ? 1 : 0);  // all the shared memory an SM has: the ring is latency-bound
  static constexpr int A_BYTES = RC_BLOCK_M * RC_BLOCK_K * 2;
  static constexpr int B_ROWS = BLOCK_N / 2;  // this CTA's half of the W' tile
  static constexpr int B_BYTES = B_ROWS * RC_BLOCK_K * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BLOCK_N;
  // barriers: full[S] (used in the even CTA), empty[S], tmem_full[2], tmem_empty[2], stats_full[2], rstd_free[2]
  // + stats_x (the four statistics warps among themselves); fused: + scores[2] (both CTAs' epilogue
  // threads), epi (the four epilogue warps among themselves)
  static constexpr int NUM_BARS = 2 * STAGES + 9 + (FUSED ? 3 : 0);
  static constexpr int BAR_BYTES = (NUM_BARS * 8 + 15) / 16 * 16;
  // fused: scores / weights [2 units][heads of the tile x FG][256 rows of the pair], 1/rms of the 256 rows
  // [2 units][256], partial sums of the weights [heads x FG][4 warps]
  static constexpr int GT = (BLOCK_N / D_HEAD) * (FUSED ? FG : 0);
  static constexpr int FUSED_BYTES = FUSED ? (2 * GT * 256 + 2 * 256 + GT * 4) * 4 : 0;
  static constexpr int LO_BYTES = LOSM ? (D_HEAD / 2) * ROPE_LO_SIZE * 8 : 0;
  static constexpr int TAIL_BYTES = BAR_BYTES + 16 /*tmem ptr, abort*/ + 2 * RC_BLOCK_M * 4 /*rstd*/ + 256 * 4 /*gamma_k*/ + FUSED_BYTES + LO_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + TAIL_BYTES;  // the base must be 1024-byte aligned
  static_assert(SMEM_BYTES <= 232448, "more shared memory than an SM offers");
};

// Optional per-tile timeline (SM clock cycles) for performance analysis; see kvd_set_trace.
template <bool TRACE>
__device__ __forceinline__ void trace_put(long long *trace, int tile_iter, int field, long long v) {
  if (TRACE && tile_iter < RC_TRACE_TILES)
    trace[(static_cast<size_t>(blockIdx.x) * RC_TRACE_TILES + tile_iter) * RC_TRACE_FIELDS + field] = v;
}
template <bool TRACE>
__device__ __forceinline__ void trace_put(long long *trace, int tile_iter, int field) {
  if (TRACE) trace_put<TRACE>(trace, tile_iter, field, clock64());
}

// The same wait with a cluster-scope acquire, for barriers whose arrivals publish data that threads of
// the partner CTA wrote.
__device__ __forceinline__ bool warp_wait_cluster(uint32_t bar, uint32_t parity, const volatile int *abort_flag,
                                                  unsigned long long timeout_ns, int lane) {
  int ok = 1;
  if (lane == 0 && !mbar_try_wait_cluster(bar, parity)) {
    const unsigned long long t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
      if (((++it) & 31u) == 0u && (*abort_flag != 0 || globaltimer_ns() - t0 > timeout_ns)) {
        ok = 0;
        break;
      }
    }
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}

// One k block (64 channels = four K=16 steps) of the pair MMA followed by the commit that frees the
// stage in both CTAs.  a_lo / b_lo are the low words of the shared-memory descriptors of the stage
// (the K step advances the start-address field by 32 bytes = 2 units); desc_hi is their common
// high word.  `acc_first` = 0 makes the first step overwrite the accumulator.
#define KVD_DEFINE_UMMA_KBLOCK(NAME, KIND) \
__device__ __forceinline__ void NAME(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, \
                                                 uint32_t idesc, uint32_t acc_first, uint32_t bar_empty) { \
  asm volatile( \
      "{\n\t" \
      ".reg .pred p, t;\n\t" \
      ".reg .b64 da, db;\n\t" \
      ".reg .b32 la, lb;\n\t" \
      "setp.ne.b32 p, %5, 0;\n\t" \
      "setp.eq.b32 t, 0, 0;\n\t" \
      "mov.b64 da, {%1, %3};\n\t" \
      "mov.b64 db, {%2, %3};\n\t" \
      "tcgen05.mma.cta_group::2.kind::" KIND " [%0], da, db, %4, p;\n\t" \
      "add.u32 la, %1, 2;\n\t" \
      "add.u32 lb, %2, 2;\n\t" \
      "mov.b64 da, {la, %3};\n\t" \
      "mov.b64 db, {lb, %3};\n\t" \
      "tcgen05.mma.cta_group::2.kind::" KIND " [%0], da, db, %4, t;\n\t" \
      "add.u32 la, %1, 4;\n\t" \
      "add.u32 lb, %2, 4;\n\t" \
      "mov.b64 da, {la, %3};\n\t" \
      "mov.b64 db, {lb, %3};\n\t" \
      "tcgen05.mma.cta_group::2.kind::" KIND " [%0], da, db, %4, t;\n\t" \
      "add.u32 la, %1, 6;\n\t" \
      "add.u32 lb, %2, 6;\n\t" \
      "mov.b64 da, {la, %3};\n\t" \
      "mov.b64 db, {lb, %3};\n\t" \
      "tcgen05.mma.cta_group::2.kind::" KIND " [%0], da, db, %4, t;\n\t" \
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%6], %7;\n\t" \
      "}" \
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first), "r"(bar_empty), \
        "h"(static_cast<uint16_t>(3)) \
      : "memory"); \
}
KVD_DEFINE_UMMA_KBLOCK(umma_kblock_pair, "f16")        // bf16 operands: 64 channels = four K=16 steps
KVD_DEFINE_UMMA_KBLOCK(umma_kblock_pair_f8, "f8f6f4")  // E4M3 operands: 128 channels = four K=32 steps
KVD_DEFINE_UMMA_KBLOCK(umma_kblock_pair_tf32, "tf32")  // fp32 operands read as TF32: 32 channels = four K=8 steps
#undef KVD_DEFINE_UMMA_KBLOCK

// Output stores.  Each epilogue thread owns one row, so the 32 lanes of a store instruction write 32
// different lines and the instruction occupies the SM's load/store data path once per lane -- cycles
// the operand ring's TMA writes and the tensor cores' operand reads compete for.  32-byte stores halve
// the instruction count, and not allocating the lines in L1 (nothing reads them back) halves the
// data-path cycles again.  `o` holds n16 * 4 packed words.
template <int N16>
__device__ __forceinline__ void store_row_piece(__nv_bfloat16 *dst, const uint32_t *o, bool wide) {
  if (wide) {
#pragma unroll
    for (int j = 0; j < N16 / 2; ++j)
      asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 16 * j),
                   "r"(o[8 * j]), "r"(o[8 * j + 1]), "r"(o[8 * j + 2]), "r"(o[8 * j + 3]), "r"(o[8 * j + 4]),
                   "r"(o[8 * j + 5]), "r"(o[8 * j + 6]), "r"(o[8 * j + 7])
                   : "memory");
  } else {
#pragma unroll
    for (int j = 0; j < N16; ++j)
      asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 8 * j), "r"(o[4 * j]),
                   "r"(o[4 * j + 1]), "r"(o[4 * j + 2]), "r"(o[4 * j + 3])
                   : "memory");
  }
}

// EB = bytes per operand element: 2 = bf16 rows and weights, 1 = the FP8 variant (E4M3 codes of rows and
// weights; a k block is then 128 channels in the same 128-byte rows, the MMA kind f8f6f4, and the rows'
// and the matrix's quantisation scales ride in the per-row factor that the statistics warps hand over).
// DT = 1: fp16 rows, weights and outputs instead of bf16 (plain variant only).
template <int BLOCK_N, int D_HEAD, bool TRACE, int FG, int EB = 2, bool LOSM = (FG > 0), int DT = 0>
__global__ void __launch_bounds__(RC_THREADS, 1)
kvd_recompute_kernel(const __grid_constant__ CUtensorMap tmap_store, const __grid_constant__ CUtensorMap tmap_rows,
                     const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ RecomputeParams p,
                     const __grid_constant__ std::conditional_t<(FG > 0), FusedParams, NoFusedParams> f) {
  using Cfg = RcCfg<BLOCK_N, D_HEAD, FG, LOSM>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr bool FUSED = FG > 0;
  static_assert(DT == 0 || (DT == 1 && EB == 2) || (DT == 2 && EB == 4 && FG == 0),
                "fp16 exists for the plain and the fused variant on 16-bit rows, fp32 for the plain variant only");
  constexpr int EW = DT == 2 ? 2 : 1;  // 16-bit units per output element (output pointers count 16-bit units)
  constexpr int KB_ELEMS = RC_BLOCK_K * 2 / EB;  // channels per k block
  static_assert(BLOCK_N % D_HEAD == 0, "a tile must hold whole heads");

  extern __shared__ __align__(1024) uint8_t smem[];
  // the 128-byte swizzle pattern is anchored at 1024-byte boundaries; there is no slack to realign
  if ((smem_u32(smem) & 1023u) != 0u) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    return;
  }
  uint8_t *tail = smem + STAGES * Cfg::STAGE_BYTES;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tail);
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(tail + Cfg::BAR_BYTES);
  volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);
  float *s_rstd = reinterpret_cast<float *>(tail + Cfg::BAR_BYTES + 16);
  float *s_gamma_k = s_rstd + 2 * RC_BLOCK_M;
  float *s_sc = s_gamma_k + 256;                 // fused: [2][GT][256]
  float *s_rall = s_sc + 2 * Cfg::GT * 256;      // fused: [2][256]
  float *s_lsum = s_rall + 2 * 256;              // fused: [GT][4]
  // LOSM: the low rotation table [pair][16], behind whatever precedes it in this variant's tail
  float2 *s_lo = reinterpret_cast<float2 *>(FUSED ? s_lsum + Cfg::GT * 4 : s_gamma_k + 256);

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto bar_full = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto bar_tmem_full = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto bar_tmem_empty = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };  // even CTA only
  auto bar_stats_full = [&](int a) { return bar_base + 8u * (2 * STAGES + 4 + a); };
  auto bar_rstd_free = [&](int a) { return bar_base + 8u * (2 * STAGES + 6 + a); };
  const uint32_t bar_stats_x = bar_base + 8u * (2 * STAGES + 8);
  auto bar_scores = [&](int u) { return bar_base + 8u * (2 * STAGES + 9 + u); };  // fused only
  const uint32_t bar_epi = bar_base + 8u * (2 * STAGES + 11);                       // fused only
  const uint32_t cta_rank = cluster_ctarank();  // 0: issues the MMAs, 1: its partner
  const int cluster_id = static_cast<int>(blockIdx.x >> 1);
  const int num_clusters = static_cast<int>(gridDim.x >> 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.num_m_blocks * p.num_n_blocks;
  // Tile order.  With more tiles than clusters a cluster works through "units" of two consecutive
  // tiles that share a row block -- the key tile and the value tile of one head column -- so that the
  // row statistics are fetched once per unit and reused; key first, so that the last tile of a CTA,
  // whose epilogue nothing overlaps, is a cheap value tile.  (Units of
  // all tiles of a row block measured slower: the units are then too few to balance the clusters.)
  // With no more tiles than clusters every tile is its own unit, all key tiles first.  Falls back to
  // row-major single tiles when a tile mixes key and value heads.
  const int nk_tiles = (p.k_cols % BLOCK_N == 0) ? p.k_cols / BLOCK_N : 0;
  // (the fused variant always pairs the key tile with the value tile: the scores of the one weight the other)
  const int unit_tiles = (nk_tiles != 0 && (FUSED || num_tiles > num_clusters)) ? 2 : 1;
  const int n_units = num_tiles / unit_tiles;
  // i-th tile of this cluster -> (job, first row of this CTA's 128 rows within the job, first fused
  // column, whether it opens a unit); false when the cluster has no i-th tile
  auto tile_at = [&](int i, int &job, int &m0, int &n0, bool &first) -> bool {
    const int unit = cluster_id + (i / unit_tiles) * num_clusters, j = i % unit_tiles;
    if (unit >= n_units) return false;
    first = j == 0;
    int mb;
    if (nk_tiles == 0) {
      mb = unit / p.num_n_blocks;
      n0 = (unit % p.num_n_blocks) * BLOCK_N;
    } else if (unit_tiles == 1) {
      if (unit < p.num_m_blocks * nk_tiles) {
        mb = unit / nk_tiles;
        n0 = (unit % nk_tiles) * BLOCK_N;
      } else {
        const int u = unit - p.num_m_blocks * nk_tiles, nv = p.num_n_blocks - nk_tiles;
        mb = u / nv;
        n0 = (nk_tiles + u % nv) * BLOCK_N;
      }
    } else {
      mb = unit / nk_tiles;
      n0 = (unit % nk_tiles + (j == 0 ? 0 : nk_tiles)) * BLOCK_N;
    }
    // jobs own consecutive runs of 256-row blocks: the last job whose first block is <= mb
    int lo = 0, hi = p.n_jobs;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (p.jobs[mid].mb_start <= mb) lo = mid;
      else hi = mid;
    }
    job = lo;
    m0 = (mb - p.jobs[lo].mb_start) * (2 * RC_BLOCK_M) + static_cast<int>(cta_rank) * RC_BLOCK_M;
    // checking build: the tile lies inside the job table, its job's row blocks and (for store ranges) the
    // sequence's slab; a tile that does not is not processed by any role
    if (!KVD_BOUNDS_OK(mb >= 0 && mb < p.num_m_blocks && lo >= 0 && lo < p.n_jobs && n0 >= 0 && n0 < p.num_n_blocks * BLOCK_N &&
                           m0 - static_cast<int>(cta_rank) * RC_BLOCK_M < p.jobs[lo].n &&
                           (p.jobs[lo].slab < 0 || p.jobs[lo].row0 + p.jobs[lo].n <= p.store_rows),
                       p.status))
      return false;
    return true;
  };
  const unsigned long long tmo = p.timeout_ns;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);   // the even CTA's producer arms it with the bytes of both CTAs
      mbar_init(bar_empty(s), 1);  // the MMA commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tmem_full(a), 1);
      mbar_init(bar_tmem_empty(a), 8);           // one arrival per epilogue warp of both CTAs
      mbar_init(bar_stats_full(a), RC_BLOCK_M);  // one arrival per statistics thread
      mbar_init(bar_rstd_free(a), 4);            // one arrival per local epilogue warp
    }
    mbar_init(bar_stats_x, 4);  // one arrival per statistics warp
    if (FUSED) {
      mbar_init(bar_scores(0), 256);  // one arrival per epilogue thread of both CTAs
      mbar_init(bar_scores(1), 256);
      mbar_init(bar_epi, 4);          // one arrival per local epilogue warp
    }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmap_store);
    prefetch_tensormap(&tmap_rows);
    prefetch_tensormap(&tmap_b);
  }
  if (threadIdx.x < D_HEAD) s_gamma_k[threadIdx.x] = p.gamma_k ? p.gamma_k[threadIdx.x] : 1.0f;
  if constexpr (LOSM) {
    // (written at kvd_set_layer time: may be read before the dependency wait below)
    const uint4 *src = reinterpret_cast<const uint4 *>(p.rope_lo);
    uint4 *dstl = reinterpret_cast<uint4 *>(s_lo);
    for (int i = threadIdx.x; i < Cfg::LO_BYTES / 16; i += RC_THREADS) dstl[i] = __ldg(src + i);
  }
  if (warp == 3) {
    tmem_alloc_pair(smem_u32(s_tmem), Cfg::TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();  // barriers of both CTAs are initialised before anyone signals across the pair
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  // The set-up above read only kernel parameters and tables written at kvd_set_layer time, so it may
  // overlap the tail of the preceding kernel; rows, positions and outputs are touched from here on.
  grid_launch_dependents();
  grid_dependency_wait();
  if (threadIdx.x == 0) {
    trace_put<TRACE>(p.trace, 0, 11);
    if (TRACE) trace_put<TRACE>(p.trace, 0, 12, static_cast<long long>(globaltimer_ns()));
  }

  if (warp == 2) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0, n_issued = 0;
      uint32_t ph = 0;
      // the stage barrier lives in the even CTA; `full` is its address as seen from this CTA
      const uint32_t full0 = map_to_cta(bar_full(0), 0);
      uint32_t full = full0, empty = bar_empty(0), dst = smem_base;
      const int b_row_off = static_cast<int>(cta_rank) * Cfg::B_ROWS;
      bool ok = true;
      int job, m0, n0;
      bool first_of_unit;
      for (int ti = 0; ok && tile_at(ti, job, m0, n0, first_of_unit); ++ti) {
        n0 += b_row_off;
        // rows come from a slab of the residual store or from the caller's buffer (slab 0 of its map)
        const int slab = p.jobs[job].slab;
        const CUtensorMap *tmap_a = slab < 0 ? &tmap_rows : &tmap_store;
        const int a_slab = slab < 0 ? 0 : slab;
        m0 += p.jobs[job].row0;
        long long waited = 0;
        trace_put<TRACE>(p.trace, ti, 1);
        for (int k0 = 0; k0 < p.num_k_blocks * KB_ELEMS; k0 += KB_ELEMS) {
          const long long w0 = TRACE ? clock64() : 0;
          if (!mbar_wait(empty, ph ^ 1u, s_abort, tmo)) {
            raise(p.status, STATUS_TIMEOUT, s_abort);
            ok = false;
            break;
          }
          if (TRACE) waited += clock64() - w0;
          if (cta_rank == 0) mbar_arrive_expect_tx(bar_full(s), 2 * Cfg::STAGE_BYTES);
          tma_load_3d_pair(dst, tmap_a, full, k0, m0, a_slab);
          tma_load_2d_pair(dst + Cfg::A_BYTES, &tmap_b, full, k0, n0);
          ++n_issued;
          full += 8u;
          empty += 8u;
          dst += Cfg::STAGE_BYTES;
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
            full = full0;
            empty = bar_empty(0);
            dst = smem_base;
          }
        }
        trace_put<TRACE>(p.trace, ti, 0, waited);
        trace_put<TRACE>(p.trace, ti, 2);
      }
      if (!ok) {
        // leave no bulk copy in flight behind us.  The even CTA waits (bounded) for every stage it
        // armed: stages below s were last filled in the current round (parity ph), the others in the
        // previous round; a stage completes only when the partner's bytes have landed too.  The odd
        // CTA cannot watch the barrier; it gives its copies a bounded time that exceeds any load
        // latency by orders of magnitude, and neither CTA leaves before the cluster barrier below.
        if (cta_rank == 0) {
          for (int i = 0; i < STAGES; ++i) {
            if (n_issued > i) {
              const uint32_t par = i < s ? ph : ph ^ 1u;
              const unsigned long long t0 = globaltimer_ns();
              while (!mbar_try_wait(bar_full(i), par)) {
                if (globaltimer_ns() - t0 > 100000000ull) break;
              }
            }
          }
        } else {
          const unsigned long long t0 = globaltimer_ns();
          while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
      }
    }
  } else if (warp == 3) {
    if (lane == 0 && cta_rank == 0) {
      // ---------------------------------------------------------------- MMA issuer (even CTA)
      constexpr uint32_t idesc = EB == 1   ? umma_idesc_e4m3_f32(2 * RC_BLOCK_M, BLOCK_N)
                                 : EB == 4 ? umma_idesc_tf32_f32(2 * RC_BLOCK_M, BLOCK_N)
                                 : DT == 1 ? umma_idesc_f16_f32(2 * RC_BLOCK_M, BLOCK_N)
                                           : umma_idesc_bf16_f32(2 * RC_BLOCK_M, BLOCK_N);
      // descriptor words for 128-byte-swizzled K-major tiles: low = start address >> 4 | LBO field (1),
      // high = SBO (1024 B >> 4) | version 1 (bit 46) | swizzle mode 2 (bits 61-63)
      constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t a_lo0 = ((smem_base & 0x3FFFFu) >> 4) | (1u << 16);
      constexpr uint32_t stage_units = Cfg::STAGE_BYTES >> 4, b_off_units = Cfg::A_BYTES >> 4;
      int s = 0, a = 0;
      uint32_t ph = 0, aph = 0;
      uint32_t full = bar_full(0), empty = bar_empty(0), a_lo = a_lo0;
      bool ok = true;
      int job_, m0_, n0_;
      bool first_;
      for (int ti = 0; ok && tile_at(ti, job_, m0_, n0_, first_); ++ti) {
        // both CTAs' epilogues have drained accumulator a
        if (!mbar_wait(bar_tmem_empty(a), aph ^ 1u, s_abort, tmo)) {
          raise(p.status, STATUS_TIMEOUT, s_abort);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BLOCK_N;
        // fused, value tile of a unit whose job attends: the operands change places, the accumulator
        // holds V transposed (lanes = the pair's 256 value channels, columns = the pair's 256 rows), so
        // that the weighted sum over rows is a sum along columns, local to a thread
        bool swap_ab = false;
        if constexpr (FUSED) swap_ab = !first_ && f.att[job_].q != nullptr;
        long long waited = 0;
        trace_put<TRACE>(p.trace, ti, 4);
        trace_put<TRACE>(p.trace, ti, 10, (m0_ / (2 * RC_BLOCK_M)) * p.num_n_blocks + n0_ / BLOCK_N);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          const long long w0 = TRACE ? clock64() : 0;
          // stage s has landed in both CTAs
          if (!mbar_wait(full, ph, s_abort, tmo)) {
            raise(p.status, STATUS_TIMEOUT, s_abort);
            ok = false;
            break;
          }
          if (TRACE) waited += clock64() - w0;
          tc_fence_after();
          if (EB == 1 && FUSED && swap_ab) umma_kblock_pair_f8(d_tmem, a_lo + b_off_units, a_lo, desc_hi, idesc, kb != 0 ? 1u : 0u, empty);
          else if (EB == 1) umma_kblock_pair_f8(d_tmem, a_lo, a_lo + b_off_units, desc_hi, idesc, kb != 0 ? 1u : 0u, empty);
          else if (EB == 4) umma_kblock_pair_tf32(d_tmem, a_lo, a_lo + b_off_units, desc_hi, idesc, kb != 0 ? 1u : 0u, empty);
          else if (FUSED && swap_ab) umma_kblock_pair(d_tmem, a_lo + b_off_units, a_lo, desc_hi, idesc, kb != 0 ? 1u : 0u, empty);
          else umma_kblock_pair(d_tmem, a_lo, a_lo + b_off_units, desc_hi, idesc, kb != 0 ? 1u : 0u, empty);
          full += 8u;
          empty += 8u;
          a_lo += stage_units;
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
            full = bar_full(0);
            empty = bar_empty(0);
            a_lo = a_lo0;
          }
        }
        if (!ok) break;
        umma_commit_pair(bar_tmem_full(a), 3);  // accumulator a is complete in both CTAs
        trace_put<TRACE>(p.trace, ti, 3, waited);
        trace_put<TRACE>(p.trace, ti, 5);
        if (++a == 2) {
          a = 0;
          aph ^= 1u;
        }
      }
    }
  } else if (warp < 2 || warp >= 8) {
    // ------------------------------------------------------------------ row statistics (Eq. 2)
    const int w4 = warp < 2 ? warp : warp - 6;  // warps 0, 1, 8, 9 -> rows 32 * w4 .. 32 * w4 + 31
    const int row = w4 * 32 + lane;
    int a = 0;
    uint32_t aph = 0;
    int job, m0, n0_;
    bool first_of_unit;
    float rstd_row = 0.f;  // of this thread's row, kept for the other tiles of the unit
    uint32_t xph = 0;      // phase of the statistics warps' own barrier
    for (int ti = 0; tile_at(ti, job, m0, n0_, first_of_unit); ++ti) {
      const long long st0 = TRACE ? clock64() : 0;
      // s_rstd[a] is free once the local epilogue that read it has finished with accumulator a
      // the whole warp takes the same branch: aligned instructions follow
      if (!warp_wait(bar_rstd_free(a), aph ^ 1u, s_abort, tmo, lane)) {
        raise(p.status, STATUS_TIMEOUT, s_abort);
        break;
      }
      if (first_of_unit) {
        const RcJob &J = p.jobs[job];
        const int n_here = J.n - m0;  // rows of this CTA's 128 that exist (may exceed 128)
        if (J.sumsq != nullptr) {
          // checkpointed rows (or caller rows whose statistics a kernel of their own took): the sum of
          // squares is read back
          const float sum = row < n_here ? __ldg(J.sumsq + m0 + row) : 0.f;
          rstd_row = 1.0f / sqrtf(sum * p.inv_d_hidden + p.rms_eps);
          // FP8 rows: the accumulator is a sum of code products; row scale and matrix scale go with 1/rms
          if (EB == 1) rstd_row *= (row < n_here ? __ldg(J.scale + m0 + row) : 0.f) * __ldg(p.w_scale);
        } else {
          // a few caller rows: the four warps share them in groups of four rows (group g -> warp g % 4),
          // leave 1/rms in s_rstd[a] and meet on a barrier before every thread picks up its own row.
          // Rows past the end of the job read the job's last row instead (no branch inside a group).
          const uint4 *base = reinterpret_cast<const uint4 *>(p.ext_rows) + static_cast<size_t>(m0) * p.row_chunks;
          // STORE_RESIDUAL in the same launch: the tile of the first column block also writes the rows it reads
          // (with their positions and statistics) into the store slots the host assigned to them
          const bool append = p.append_n > 0 && n0_ == 0;
#pragma unroll 1
          for (int g = w4; g < 32 && 4 * g < n_here; g += 4) {
            const uint4 *src[4];
            uint4 *dst[4] = {nullptr, nullptr, nullptr, nullptr};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int r = 4 * g + i;
              src[i] = base + static_cast<size_t>(r < n_here ? r : n_here - 1) * p.row_chunks;
              if (append && r < n_here && m0 + r < p.append_n)
                dst[i] = p.append_rows + static_cast<size_t>(p.append_slot[m0 + r]) * p.row_chunks;
            }
            float ss[4];
            if (append) warp_rows_sumsq<4, 4, true, DT>(src, dst, p.row_chunks, lane, ss);
            else warp_rows_sumsq<4, 4, false, DT>(src, dst, p.row_chunks, lane, ss);
            const float mine = lane == 0 ? ss[0] : lane == 1 ? ss[1] : lane == 2 ? ss[2] : ss[3];
            if (lane < 4 && 4 * g + lane < n_here) {
              s_rstd[a * RC_BLOCK_M + 4 * g + lane] = 1.0f / sqrtf(mine * p.inv_d_hidden + p.rms_eps);
              if (append && m0 + 4 * g + lane < p.append_n) {
                const long long slot = p.append_slot[m0 + 4 * g + lane];
                p.append_sumsq[slot] = mine;
                p.append_pos[slot] = J.positions[m0 + 4 * g + lane];
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_stats_x);
          if (!warp_wait(bar_stats_x, xph, s_abort, tmo, lane)) {
            raise(p.status, STATUS_TIMEOUT, s_abort);
            break;
          }
          xph ^= 1u;
          rstd_row = row < n_here ? s_rstd[a * RC_BLOCK_M + row] : 0.f;
        }
      }
      s_rstd[a * RC_BLOCK_M + row] = rstd_row;
      mbar_arrive(bar_stats_full(a));
      if (TRACE && threadIdx.x == 0) {
        trace_put<TRACE>(p.trace, ti, 8, 0);
        trace_put<TRACE>(p.trace, ti, 9, clock64() - st0);
      }
      if (++a == 2) {
        a = 0;
        aph ^= 1u;
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int row = quarter * 32 + lane;
    const uint32_t lane_field = static_cast<uint32_t>(quarter * 32) << 16;
    constexpr int HALF = D_HEAD / 2;
    constexpr int NG = FUSED ? FG : 1;
    int a = 0;
    uint32_t aph = 0;
    uint32_t sph[2] = {0u, 0u}, eph = 0;  // fused: phases of the score barriers and of the epilogue warps' barrier
    int job, m0, n0;
    bool first_of_unit;
    for (int ti = 0; tile_at(ti, job, m0, n0, first_of_unit); ++ti) {
      const RcJob &J = p.jobs[job];
      // fused: does this tile's job attend (K and V are consumed here) or is it a plain job?
      bool attend = false;
      int q_pos = 0, lo_pos = 0, part_base = 0;
      const __nv_bfloat16 *qrow = nullptr;
      if constexpr (FUSED) {
        const RcAttend &A = f.att[job];
        attend = A.q != nullptr;
        qrow = A.q;
        q_pos = A.q_pos;
        lo_pos = A.lo_pos;
        part_base = A.part_base;
      }
      const int ubuf = (ti >> 1) & 1;  // fused: score buffer of this unit
      float f_scale = 0.f;
      if constexpr (FUSED) f_scale = f.scale_log2e;
      // warp-uniform outcome: tcgen05.ld below is an aligned instruction
      if (!warp_wait(bar_tmem_full(a), aph, s_abort, tmo, lane) || !warp_wait(bar_stats_full(a), aph, s_abort, tmo, lane)) {
        raise(p.status, STATUS_TIMEOUT, s_abort);
        break;
      }
      tc_fence_after();
      if (TRACE && threadIdx.x == 4 * 32) trace_put<TRACE>(p.trace, ti, 6);
      const int m = m0 + row;
      const bool valid = m < J.n;
      const bool wide = p.wide_store != 0;
      const long long out_stride = J.slab < 0 ? p.rows_out_stride : p.out_row_stride;  // the caller's rows may go elsewhere
      const float rstd = s_rstd[a * RC_BLOCK_M + row];
      int pos = valid ? J.positions[m] : 0;
      if (pos < 0 || pos >= p.max_pos) {
        atomicOr(p.status, STATUS_POSITION);
        pos = pos < 0 ? 0 : p.max_pos - 1;
      }
      // (cos, sin) of pos * f_i = angle sum of the entries for (pos & ~15) [shared by 16 neighbouring
      // positions] and (pos & 15) [laid out [pair][low bits]: the 32 rows of a warp read one 128-byte
      // line per pair, which stays in L1]
      const float4 *t_hi = reinterpret_cast<const float4 *>(p.rope_hi + static_cast<size_t>(pos >> ROPE_LO_BITS) * HALF);
      const float2 *t_lo = (LOSM ? static_cast<const float2 *>(s_lo) : p.rope_lo) + (pos & (ROPE_LO_SIZE - 1));
      const uint32_t acc = tmem_base + lane_field + a * BLOCK_N;
      const bool visible = valid && pos <= q_pos && pos >= lo_pos;  // fused: does the query see this row's key
      bool ok = true;

      if (FUSED && attend && !first_of_unit) {
        // ---- fused, value tile (Eq. 14 into Eq. 7): the accumulator holds V transposed and unscaled --
        // this thread's lane is value channel ch of the 256-wide tile, column r is row r of the pair's
        // 256 rows.  out[ch] = sum_r w[r] * acc[ch][r] with w[r] = exp2(score[r] - max) / rms(x_r).
        constexpr int GT = Cfg::GT;
        constexpr int WPH = D_HEAD >= 128 ? 4 : D_HEAD / 32;  // local epilogue warps that share a head
        constexpr int RPW = 256 / WPH;                          // rows whose weights each of them makes
        const int ch = static_cast<int>(cta_rank) * RC_BLOCK_M + row;
        const int hh = ch / D_HEAD, cih = ch % D_HEAD, wi = quarter % WPH;
        float *sc = s_sc + (ubuf * GT + hh * NG) * 256;
        const float *ra = s_rall + ubuf * 256;
        auto epi_sync = [&]() -> bool {
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_epi);
          const bool good = warp_wait(bar_epi, eph, s_abort, tmo, lane);
          eph ^= 1u;
          return good;
        };
        // the scores and 1/rms of all 256 rows (both CTAs' key-tile epilogues) have arrived
        if (!warp_wait_cluster(bar_scores(ubuf), sph[ubuf], s_abort, tmo, lane)) {
          raise(p.status, STATUS_TIMEOUT, s_abort);
          break;
        }
        sph[ubuf] ^= 1u;
        float mx[NG], lsum[NG], o[NG];
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          float mv = -CUDART_INF_F;
#pragma unroll
          for (int k = 0; k < 8; ++k) mv = fmaxf(mv, sc[g * 256 + lane + 32 * k]);
#pragma unroll
          for (int msk = 16; msk >= 1; msk >>= 1) mv = fmaxf(mv, __shfl_xor_sync(0xffffffffu, mv, msk));
          mx[g] = mv;
        }
        if (!epi_sync()) {  // every warp has its maxima before the scores become weights
          raise(p.status, STATUS_TIMEOUT, s_abort);
          break;
        }
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          float lp = 0.f;
#pragma unroll
          for (int k = 0; k < RPW / 32; ++k) {
            const int r = wi * RPW + lane + 32 * k;
            const float pw = mx[g] == -CUDART_INF_F ? 0.f : exp2f(sc[g * 256 + r] - mx[g]);
            lp += pw;
            sc[g * 256 + r] = pw * ra[r];
          }
#pragma unroll
          for (int msk = 16; msk >= 1; msk >>= 1) lp += __shfl_xor_sync(0xffffffffu, lp, msk);
          if (lane == 0) s_lsum[(hh * NG + g) * 4 + wi] = lp;
        }
        if (!epi_sync()) {
          raise(p.status, STATUS_TIMEOUT, s_abort);
          break;
        }
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          float l = 0.f;
#pragma unroll
          for (int w = 0; w < WPH; ++w) l += s_lsum[(hh * NG + g) * 4 + w];
          lsum[g] = l;
          o[g] = 0.f;
        }
        // rows past the end of the job hold whatever the store holds there (possibly NaN patterns):
        // their weight is zero, but 0 * NaN is not, so those columns are skipped or zeroed
        const int nvalid = J.n - (m0 - static_cast<int>(cta_rank) * RC_BLOCK_M);
#pragma unroll 1
        for (int c8 = 0; c8 < 8 && c8 * 32 < nvalid; ++c8) {
          uint32_t r[32];
          tmem_ld_x32(acc + c8 * 32, r);
          tmem_wait_ld();
          if (c8 * 32 + 32 > nvalid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c8 * 32 + j >= nvalid) r[j] = 0u;
          }
#pragma unroll
          for (int g = 0; g < NG; ++g) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 w4 = *reinterpret_cast<const float4 *>(sc + g * 256 + c8 * 32 + j);
              o[g] = fmaf(w4.x, __uint_as_float(r[j]), o[g]);
              o[g] = fmaf(w4.y, __uint_as_float(r[j + 1]), o[g]);
              o[g] = fmaf(w4.z, __uint_as_float(r[j + 2]), o[g]);
              o[g] = fmaf(w4.w, __uint_as_float(r[j + 3]), o[g]);
            }
          }
        }
        if constexpr (FUSED) {
          const size_t slot = static_cast<size_t>(part_base) + (m0 - static_cast<int>(cta_rank) * RC_BLOCK_M) / (2 * RC_BLOCK_M);
          const int kvh = (n0 - p.k_cols) / D_HEAD + hh;
#pragma unroll
          for (int g = 0; g < NG; ++g) {
            const size_t qh = slot * f.n_q + static_cast<size_t>(kvh) * NG + g;
            f.part_o[qh * D_HEAD + cih] = o[g];
            if (cih == 0) *reinterpret_cast<float2 *>(f.part_ml + qh * 2) = make_float2(mx[g], lsum[g]);
          }
        }
      } else {

#pragma unroll 1
      for (int hh = 0; hh < BLOCK_N / D_HEAD; ++hh) {
        const int col0 = n0 + hh * D_HEAD;  // first fused column of this head
        const uint32_t tcol = acc + hh * D_HEAD;
        if (col0 >= p.k_cols) {
          // ---- value head (Eq. 14): scale by 1/rms and store
          __nv_bfloat16 *dst = J.v_out + (static_cast<size_t>(m) * out_stride + (col0 - p.k_cols)) * EW;
#pragma unroll 1
          for (int c = 0; c < D_HEAD / 32; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tcol + c * 32, r);
            tmem_wait_ld();
            uint32_t o[16 * EW];
#pragma unroll
            for (int j = 0; j < 16; ++j)
              emit_pair<DT>(o, j, __uint_as_float(r[2 * j]) * rstd, __uint_as_float(r[2 * j + 1]) * rstd);
            if (valid) store_row_piece<4 * EW>(dst + c * 32 * EW, o, wide);
          }
        } else {
          // ---- key head (Eq. 13): 1/rms, optional key norm, rotation R_pos
          __nv_bfloat16 *dst = J.k_out + (static_cast<size_t>(m) * out_stride + col0) * EW;
          float kscale = rstd;
          // fused, attending job: the rotated key (rounded to bf16 like a stored one) is not written but
          // multiplied with the NG queries of this KV head (Eq. 6); two-wide partial sums per query
          uint64_t sdot[NG];
#pragma unroll
          for (int g = 0; g < NG; ++g) sdot[g] = 0ull;
          const uint4 *qh = nullptr;  // the queries of this KV head: [NG][D_HEAD] bf16
          if (FUSED && attend) qh = reinterpret_cast<const uint4 *>(qrow + static_cast<size_t>(col0 / D_HEAD) * NG * D_HEAD);
          if (p.qk_norm) {
            // sum of squares over the head in four chains (columns j mod 4), two-wide, combined in a
            // fixed order: a single 256-long dependent chain would be pure latency
            uint64_t ss2[2] = {0ull, 0ull};
            const uint64_t rstd2 = pack2(rstd, rstd);
#pragma unroll 1
            for (int c = 0; c < D_HEAD / 32; ++c) {
              uint32_t r[32];
              tmem_ld_x32(tcol + c * 32, r);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                const uint64_t v0 = fmul2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), rstd2);
                const uint64_t v1 = fmul2(pack2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), rstd2);
                ss2[0] = ffma2(v0, v0, ss2[0]);
                ss2[1] = ffma2(v1, v1, ss2[1]);
              }
            }
            float s0, s1, s2, s3;
            unpack2(ss2[0], s0, s1);
            unpack2(ss2[1], s2, s3);
            const float ss = (s0 + s1) + (s2 + s3);
            kscale = rstd * (1.0f / sqrtf(ss * (1.0f / D_HEAD) + p.qk_eps));
          }
          if (p.rope_style == KVD_ROPE_INTERLEAVED) {
            constexpr int NC = D_HEAD / 16;  // 16 columns = 8 rotation pairs per step
            float4 hn[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) hn[j] = t_hi[j];
#pragma unroll 1
            for (int c = 0; c < NC; ++c) {
              float4 h[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) h[j] = hn[j];
              const int cn = c + 1 < NC ? c + 1 : c;  // prefetch the next step's table entries
#pragma unroll
              for (int j = 0; j < 4; ++j) hn[j] = t_hi[cn * 4 + j];
              uint32_t r[16];
              tmem_ld_x16(tcol + c * 16, r);
              tmem_wait_ld();
              uint32_t o[8 * EW];
#pragma unroll
              for (int j = 0; j < 8; j += 2) {
                const int i = c * 8 + j;  // pairs i and i + 1
                const float2 l0 = LOSM ? t_lo[i * ROPE_LO_SIZE] : __ldg(t_lo + i * ROPE_LO_SIZE), l1 = LOSM ? t_lo[(i + 1) * ROPE_LO_SIZE] : __ldg(t_lo + (i + 1) * ROPE_LO_SIZE);
                const float4 hh4 = h[j >> 1];
                const float c0 = fmaf(hh4.x, l0.x, -hh4.y * l0.y), s0 = fmaf(hh4.y, l0.x, hh4.x * l0.y);
                const float c1 = fmaf(hh4.z, l1.x, -hh4.w * l1.y), s1 = fmaf(hh4.w, l1.x, hh4.z * l1.y);
                const float a0 = __uint_as_float(r[2 * j]) * kscale * s_gamma_k[c * 16 + 2 * j];
                const float b0 = __uint_as_float(r[2 * j + 1]) * kscale * s_gamma_k[c * 16 + 2 * j + 1];
                const float a1 = __uint_as_float(r[2 * j + 2]) * kscale * s_gamma_k[c * 16 + 2 * j + 2];
                const float b1 = __uint_as_float(r[2 * j + 3]) * kscale * s_gamma_k[c * 16 + 2 * j + 3];
                emit_pair<DT>(o, j, fmaf(a0, c0, -b0 * s0), fmaf(a0, s0, b0 * c0));
                emit_pair<DT>(o, j + 1, fmaf(a1, c1, -b1 * s1), fmaf(a1, s1, b1 * c1));
              }
              if (FUSED && attend) {
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                  const uint4 q0 = __ldg(qh + (g * D_HEAD + c * 16) / 8), q1 = __ldg(qh + (g * D_HEAD + c * 16) / 8 + 1);
                  const uint32_t qw[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
                  for (int w = 0; w < 8; ++w) sdot[g] = ffma2(x2_to_f32x2<DT>(o[w]), x2_to_f32x2<DT>(qw[w]), sdot[g]);
                }
              } else if (valid) {
                store_row_piece<2 * EW>(dst + c * 16 * EW, o, wide);
              }
            }
          } else {
            constexpr int NC = HALF / 16;  // 16 pairs (i, i + HALF) per step
            float4 hn[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) hn[j] = t_hi[j];
#pragma unroll 1
            for (int c = 0; c < NC; ++c) {
              float4 h[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) h[j] = hn[j];
              const int cn = c + 1 < NC ? c + 1 : c;
#pragma unroll
              for (int j = 0; j < 8; ++j) hn[j] = t_hi[cn * 8 + j];
              uint32_t ra[16], rb[16];
              tmem_ld_x16(tcol + c * 16, ra);
              tmem_ld_x16(tcol + HALF + c * 16, rb);
              tmem_wait_ld();
              uint32_t oa[8 * EW], ob[8 * EW];
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                const int i = c * 16 + j;  // pairs (i, i + HALF) and (i + 1, i + 1 + HALF)
                const float2 l0 = LOSM ? t_lo[i * ROPE_LO_SIZE] : __ldg(t_lo + i * ROPE_LO_SIZE), l1 = LOSM ? t_lo[(i + 1) * ROPE_LO_SIZE] : __ldg(t_lo + (i + 1) * ROPE_LO_SIZE);
                const float4 hh4 = h[j >> 1];
                const float c0 = fmaf(hh4.x, l0.x, -hh4.y * l0.y), s0 = fmaf(hh4.y, l0.x, hh4.x * l0.y);
                const float c1 = fmaf(hh4.z, l1.x, -hh4.w * l1.y), s1 = fmaf(hh4.w, l1.x, hh4.z * l1.y);
                const float a0 = __uint_as_float(ra[j]) * kscale * s_gamma_k[i];
                const float b0 = __uint_as_float(rb[j]) * kscale * s_gamma_k[i + HALF];
                const float a1 = __uint_as_float(ra[j + 1]) * kscale * s_gamma_k[i + 1];
                const float b1 = __uint_as_float(rb[j + 1]) * kscale * s_gamma_k[i + 1 + HALF];
                emit_pair<DT>(oa, j >> 1, fmaf(a0, c0, -b0 * s0), fmaf(a1, c1, -b1 * s1));
                emit_pair<DT>(ob, j >> 1, fmaf(a0, s0, b0 * c0), fmaf(a1, s1, b1 * c1));
              }
              if (FUSED && attend) {
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                  const uint4 a0 = __ldg(qh + (g * D_HEAD + c * 16) / 8), a1 = __ldg(qh + (g * D_HEAD + c * 16) / 8 + 1);
                  const uint4 b0 = __ldg(qh + (g * D_HEAD + HALF + c * 16) / 8), b1 = __ldg(qh + (g * D_HEAD + HALF + c * 16) / 8 + 1);
                  const uint32_t qa[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                  const uint32_t qb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                  for (int w = 0; w < 8; ++w) {
                    sdot[g] = ffma2(x2_to_f32x2<DT>(oa[w]), x2_to_f32x2<DT>(qa[w]), sdot[g]);
                    sdot[g] = ffma2(x2_to_f32x2<DT>(ob[w]), x2_to_f32x2<DT>(qb[w]), sdot[g]);
                  }
                }
              } else if (valid) {
                store_row_piece<2 * EW>(dst + c * 16 * EW, oa, wide);
                store_row_piece<2 * EW>(dst + (HALF + c * 16) * EW, ob, wide);
              }
            }
          }
          if (FUSED && attend) {
            // the scores of this row (log2 units, -inf when the query does not see the key) go to both
            // CTAs of the pair: the value tile's epilogue needs those of all 256 rows
#pragma unroll
            for (int g = 0; g < NG; ++g) {
              float lo, hi;
              unpack2(sdot[g], lo, hi);
              float sv = (lo + hi) * f_scale;
              if (!visible) sv = -CUDART_INF_F;
              float *dstp = s_sc + (ubuf * Cfg::GT + hh * NG + g) * 256 + static_cast<int>(cta_rank) * RC_BLOCK_M + row;
              *dstp = sv;
              st_cluster_f32(map_to_cta(smem_u32(dstp), cta_rank ^ 1u), sv);
            }
          }
        }
      }
      if (FUSED && attend) {
        // 1/rms of the row, then "this thread's scores are in place" to both CTAs (a release at cluster
        // scope: the partner's value-tile epilogue reads what was just stored into its shared memory)
        float *rp = s_rall + ubuf * 256 + static_cast<int>(cta_rank) * RC_BLOCK_M + row;
        *rp = rstd;
        st_cluster_f32(map_to_cta(smem_u32(rp), cta_rank ^ 1u), rstd);
        mbar_arrive(bar_scores(ubuf));
        mbar_arrive_cluster_release(map_to_cta(bar_scores(ubuf), cta_rank ^ 1u));
      }
      }
      if (!ok) break;
      // accumulator a (and s_rstd[a]) may be overwritten now
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar_rstd_free(a));
        if (cta_rank == 0) mbar_arrive(bar_tmem_empty(a));
        else mbar_arrive_cluster(map_to_cta(bar_tmem_empty(a), 0));
      }
      if (TRACE && threadIdx.x == 4 * 32) trace_put<TRACE>(p.trace, ti, 7);
      if (++a == 2) {
        a = 0;
        aph ^= 1u;
      }
    }
  }

  // nobody may leave while the partner can still signal into this CTA's shared memory
  tc_fence_before();
  cluster_sync_all();
  if (TRACE && threadIdx.x == 0) {
    trace_put<TRACE>(p.trace, 0, 13, static_cast<long long>(globaltimer_ns()));
    trace_put<TRACE>(p.trace, 0, 14);
  }
  if (warp == 3) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------ host launcher
template <int BLOCK_N, int D_HEAD, bool TRACE, int FG, int EB = 2, bool LOSM = (FG > 0), int DT = 0>
static kvd_status launch_impl(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                              const CUtensorMap &tmap_rows, const RecomputeParams &p, const FusedParams *fp,
                              cudaStream_t stream) {
  using Cfg = RcCfg<BLOCK_N, D_HEAD, FG, LOSM>;
  auto kern = kvd_recompute_kernel<BLOCK_N, D_HEAD, TRACE, FG, EB, LOSM, DT>;
  const CUtensorMap &tmap_b = EB == 1 ? ls.tmap_b8 : ls.tmap_b;
  static bool configured[64] = {};
  if (!configured[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(recompute)");
    configured[ctx->device & 63] = true;
  }
  // plain: one cluster per tile at most; fused: per unit of a key tile and a value tile
  const int work = FG > 0 ? p.num_m_blocks * p.num_n_blocks / 2 : p.num_m_blocks * p.num_n_blocks;
  const int max_clusters = ctx->num_sms / 2;
  const int clusters = work < max_clusters ? work : max_clusters;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2 * clusters, 1, 1);
  cfg.blockDim = dim3(RC_THREADS, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = (serial_launch_mask() & 1) ? 0 : 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t le;
  if constexpr (FG > 0) le = cudaLaunchKernelEx(&cfg, kern, tmap_store, tmap_rows, tmap_b, p, *fp);
  else le = cudaLaunchKernelEx(&cfg, kern, tmap_store, tmap_rows, tmap_b, p, NoFusedParams());
  if (le != cudaSuccess) return cuda_fail(ctx, le, "launch recompute");
  ctx->launches += 1;
  return KVD_OK;
}

template <int BLOCK_N, int D_HEAD, int FG = 0>
static kvd_status launch_sel(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                             const CUtensorMap &tmap_rows, const RecomputeParams &p, const FusedParams *fp,
                             cudaStream_t stream) {
  if constexpr (FG == 0) {
    // fp16 and fp32 contexts: one variant (low table in shared memory) for all launch sizes
    if (ctx->dtype == 1) return launch_impl<BLOCK_N, D_HEAD, false, 0, 2, true, 1>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
    if (ctx->dtype == 2) return launch_impl<BLOCK_N, D_HEAD, false, 0, 4, true, 2>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
    if (p.trace != nullptr) return launch_impl<BLOCK_N, D_HEAD, true, 0>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
    // one tile per cluster at most: every key tile's epilogue is exposed -> the low table from shared memory
    if (p.num_m_blocks * p.num_n_blocks <= ctx->num_sms / 2)
      return launch_impl<BLOCK_N, D_HEAD, false, 0, 2, true>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
  }
  // the fused variant on fp16 rows, weights, queries and outputs (same tiles, MMA kind f16 with fp16 operands)
  if constexpr (FG > 0) {
    if (ctx->dtype == 1) return launch_impl<BLOCK_N, D_HEAD, false, FG, 2, true, 1>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
  }
  return launch_impl<BLOCK_N, D_HEAD, false, FG>(ctx, ls, tmap_store, tmap_rows, p, fp, stream);
}

kvd_status launch_recompute(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                            const CUtensorMap &tmap_rows, const RecomputeParams &p, cudaStream_t stream) {
  const int dh = ctx->desc.d_head;
  if (ctx->block_n == 256) {
    if (dh == 256) return launch_sel<256, 256>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 128) return launch_sel<256, 128>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 64) return launch_sel<256, 64>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
  } else if (ctx->block_n == 128) {
    if (dh == 128) return launch_sel<128, 128>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 64) return launch_sel<128, 64>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
  }
  return KVD_ERR_SHAPE;
}

// The fused variant exists for 256-column tiles and the head sizes / group sizes of the model shapes
// this library is built around; KVD_ERR_UNSUPPORTED otherwise (the caller falls back to
// kvd_recompute_kv + kvd_decode_attention).
kvd_status launch_recompute_fused(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                                  const CUtensorMap &tmap_rows, const RecomputeParams &p, const FusedParams &fp,
                                  cudaStream_t stream, int eb) {
  const int dh = ctx->desc.d_head, g = ctx->desc.n_q_heads / ctx->desc.n_kv_heads;
  if (ctx->block_n != 256 || p.k_cols % 256 != 0) return KVD_ERR_UNSUPPORTED;
  if (eb == 1) {  // rows and weights as E4M3 codes (the FP8 store)
    if (dh == 256 && g == 2 && p.trace != nullptr) return launch_impl<256, 256, true, 2, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    if (dh == 256 && g == 2) return launch_impl<256, 256, false, 2, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    if (dh == 256 && g == 1) return launch_impl<256, 256, false, 1, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    if (dh == 128 && g == 4) return launch_impl<256, 128, false, 4, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    if (dh == 128 && g == 2) return launch_impl<256, 128, false, 2, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    if (dh == 128 && g == 1) return launch_impl<256, 128, false, 1, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
    return KVD_ERR_UNSUPPORTED;
  }
  if (dh == 256 && g == 2) return launch_sel<256, 256, 2>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
  if (dh == 256 && g == 1) return launch_sel<256, 256, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
  if (dh == 128 && g == 4) return launch_sel<256, 128, 4>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
  if (dh == 128 && g == 2) return launch_sel<256, 128, 2>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
  if (dh == 128 && g == 1) return launch_sel<256, 128, 1>(ctx, ls, tmap_store, tmap_rows, p, &fp, stream);
  return KVD_ERR_UNSUPPORTED;
}

// The FP8 variant: rows and weights as E4M3 codes (tmap_store is the FP8 store's map, tmap_rows the map of
// the caller's quantised rows, or the store's again).
kvd_status launch_recompute_fp8(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                                const CUtensorMap &tmap_rows, const RecomputeParams &p, cudaStream_t stream) {
  const int dh = ctx->desc.d_head;
  if (ctx->block_n == 256) {
    if (dh == 256 && p.trace != nullptr) return launch_impl<256, 256, true, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 256) return launch_impl<256, 256, false, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 128) return launch_impl<256, 128, false, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 64) return launch_impl<256, 64, false, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
  } else if (ctx->block_n == 128) {
    if (dh == 128) return launch_impl<128, 128, false, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
    if (dh == 64) return launch_impl<128, 64, false, 0, 1, true>(ctx, ls, tmap_store, tmap_rows, p, nullptr, stream);
  }
  return KVD_ERR_SHAPE;
}

}  // namespace kvd
