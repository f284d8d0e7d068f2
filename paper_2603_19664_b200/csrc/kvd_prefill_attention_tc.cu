// ATTENTION of Algorithm 1 (Eq. 6-7) for many query tokens of one sequence on the fifth-generation tensor cores.
//
//   CTA   = (tile of query tokens, KV head): 128 MMA rows = 128 / G tokens x the G query heads of the head's group (for
//           G = 3, 42 tokens and two empty rows; empty rows are zeros that are never stored).
//   pair  = for d_head >= 128 two CTAs with neighbouring tiles of the same KV head form a cluster and run the products
//           as tcgen05.mma.cta_group::2 (M = 256, 128 rows per CTA): a K or V block is shared by the pair, each CTA
//           loads and holds half of it (K: half the keys, V: half the channels -- the halves the instruction reads from
//           either shared memory).  Half the bytes per CTA through L2 and shared memory, twice the blocks in flight.
//   keys  = blocks of 64, aligned to ABSOLUTE position, walked in ascending order from the first block any row of the
//           pair can see to the last one.
//   TMEM  = [ O : d_head columns | S_0, S_1 : 64 columns each | Q : d_head / 2 columns ].  The query tile is written
//           there once (two elements per 32-bit column) and is the A operand of S_j = Q K_j^T; the softmax threads
//           read S_j (one row per thread, no shuffles) and hand its columns back at once (scores that are free early
//           let S run two blocks ahead); the weights P_j, in the element type, are the A operand of O += P_j V_j --
//           from 2 x 32 more columns of tensor memory for d_head <= 128, from shared memory at 256, where tensor
//           memory is full.
//   warps = 0-7 softmax and epilogue (two groups of four, TMEM lane quarter = warp % 4, alternating blocks), 8 issues
//           the S products, 9 the PV products (in the pair's leading CTA only), 10-13 gather K/V blocks from the
//           segments with 16-byte cp.async into the 128-byte-swizzled layouts the two products expect (K block:
//           K-major B operand, rows = keys; V block: the same bytes read as an MN-major B operand, rows = the
//           contraction index), a ring of K blocks and a ring of V blocks.  Positions no segment holds are
//           zero-filled and masked.
//   order = S_j is issued as soon as its K block has landed and the softmax threads have read S_{j-2} out of its
//           columns, so the scores run up to two blocks ahead of the softmax; PV_j follows the softmax of block j.  O is
//           rescaled in tensor memory only when a row of the warp moves its reference maximum (the others multiply by
//           exactly 1), and a row moves it only when a block's maximum exceeds it by a factor of 256: with exact maxima
//           some row of a 128-row tile moves in nearly every block, and rescale -> PV_j -> rescale is a serial chain.
//
// A row's result depends on that row alone: the rows of an MMA are computed independently, every row walks the key
// blocks in ascending order, a block without a visible key for the row changes nothing for it (weights 0, rescale by
// exactly 1, O += 0), and the block boundaries are absolute.  So a token attended alone and the same token inside any
// tile give the same bits.  They are not the bits of kvd_decode_attention (another split of the keys, P rounded before
// the second product).  Every wait is bounded: on a timeout the CTA raises the status word, all roles leave their
// loops, and tensor memory is freed.
#include <math_constants.h>
#include <stdlib.h>
#include <string.h>

#include <type_traits>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

constexpr int PT_ROWS = 128;     // MMA rows per CTA
constexpr int PT_KEYS = 64;      // keys per block
constexpr int PT_THREADS = 448;  // fourteen warps
constexpr int PT_LOADERS = 128;  // threads of warps 10-13
constexpr float PT_TAU = 8.0f;   // log2 of the largest weight a row may reach before its reference maximum moves
constexpr int PT_LAG = 3;        // blocks a loader thread keeps in flight behind the one it is issuing

template <int D_HEAD, bool PAIR>
struct PtCfg {
  static constexpr int NCTA = PAIR ? 2 : 1;
  static constexpr int K_ROWS = PT_KEYS / NCTA;                   // keys of a block this CTA holds
  static constexpr int V_COLS = D_HEAD / NCTA;                    // channels of a block this CTA holds
  static constexpr int TILE_BYTES = PT_KEYS * D_HEAD * 2 / NCTA;  // this CTA's share of one K or V block
  static constexpr int SLAB_K = K_ROWS * 128;                     // 64 channels of this CTA's keys
  static constexpr int SLAB_V = PT_KEYS * 128;                    // 64 of this CTA's channels of every key
  static constexpr int SLOTS_K = D_HEAD == 256 ? (PAIR ? 6 : 3) : (PAIR ? 6 : 4);  // blocks in the K ring (the scores run ahead)
  static constexpr int SLOTS_V = D_HEAD == 256 ? (PAIR ? 4 : 2) : (PAIR ? 6 : 4);  // blocks in the V ring
  static constexpr int SLOTS = SLOTS_K + SLOTS_V;
  static constexpr int COL_O = 0, COL_S = D_HEAD, COL_Q = D_HEAD + 2 * PT_KEYS;
  static constexpr bool P_TMEM = D_HEAD <= 128;                   // room for the weights in tensor memory as well
  static constexpr int COL_P = COL_Q + D_HEAD / 2;                // two blocks of weights, 32 columns each (P_TMEM)
  static constexpr int COLS_USED = COL_P + (P_TMEM ? PT_KEYS : 0);
  static constexpr int COLS = COLS_USED <= 256 ? 256 : 512;       // allocation: a power of two
  static constexpr int P_BYTES = P_TMEM ? 0 : PT_ROWS * PT_KEYS * 2;  // one block of weights in shared memory otherwise
  static constexpr int N_BARS = 2 * SLOTS + 22;
  static constexpr int SMEM_BYTES = 1024 + SLOTS * TILE_BYTES + 2 * P_BYTES + N_BARS * 8;
};

// A wait of this kernel.  Every SM sub-partition hosts a warp of either softmax group, a loader warp and possibly an MMA
// thread, and at any time some of them wait: a short sleep between polls leaves the issue slots to the warps that
// compute (+2 to 7 %).  In a pair
// the arrivals may come from the partner CTA and publish what its threads wrote to its own shared memory, so the
// acquire is at cluster scope there.
template <bool CLUSTER>
__device__ __forceinline__ bool polite_wait(uint32_t bar, uint32_t parity, const volatile int *abort_flag, unsigned long long timeout_ns) {
  auto done = [&]() { return CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
  if (done()) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t it = 0;
  while (!done()) {
    __nanosleep(20);
    if (((++it) & 31u) == 0u && (*abort_flag != 0 || globaltimer_ns() - t0 > timeout_ns)) return false;
  }
  return true;
}
// The same for a whole warp: lane 0 waits, the result is broadcast.
__device__ __forceinline__ bool polite_warp_wait(uint32_t bar, uint32_t parity, const volatile int *abort_flag, unsigned long long timeout_ns, int lane) {
  int ok = 1;
  if (lane == 0) ok = polite_wait<false>(bar, parity, abort_flag, timeout_ns) ? 1 : 0;
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}
template <bool PAIR>
__device__ __forceinline__ bool lead_wait(uint32_t bar, uint32_t parity, const volatile int *abort_flag, unsigned long long timeout_ns) {
  return polite_wait<PAIR>(bar, parity, abort_flag, timeout_ns);
}

template <int D_HEAD, int G, int DT, bool PAIR>
__global__ void __launch_bounds__(PT_THREADS, 1) kvd_prefill_attn_tc_kernel(const __grid_constant__ PrefillParams P) {
  using Cfg = PtCfg<D_HEAD, PAIR>;
  constexpr int TOK = PT_ROWS / G;     // query tokens per CTA (G = 3: 42 tokens, the last two MMA rows stay empty)
  constexpr int NCTA = Cfg::NCTA;
  constexpr int SLOTS = Cfg::SLOTS, SLOTS_K = Cfg::SLOTS_K, SLOTS_V = Cfg::SLOTS_V;
  extern __shared__ uint8_t pt_smem_raw[];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort_i, s_lo, s_hi;
  __shared__ float s_mx[2][PT_ROWS], s_lx[2][PT_ROWS];  // per group: the row maximum after its last block, its part of the row sum
  volatile int *s_abort = &s_abort_i;
  // the rings start on a 1024-byte boundary (the swizzle is a function of the address), the barriers follow them
  const uint32_t ring = (smem_u32(pt_smem_raw) + 1023u) & ~1023u;
  const uint32_t ring_v = ring + SLOTS_K * Cfg::TILE_BYTES;  // K blocks first, V blocks behind them
  const uint32_t p_smem = ring + SLOTS * Cfg::TILE_BYTES;    // two blocks of weights
  const uint32_t bar_base = p_smem + 2 * Cfg::P_BYTES;
  // barriers the MMA threads wait on are used in the leading CTA only; the others (MMA commits) in both
  auto bar_full = [&](int v, int s) { return bar_base + 8u * (v * SLOTS_K + s); };           // leader: a block has landed
  auto bar_empty = [&](int v, int s) { return bar_base + 8u * (SLOTS + v * SLOTS_K + s); };  // both: its product is done
  auto bar_s_full = [&](int b) { return bar_base + 8u * (2 * SLOTS + b); };                  // both: scores of a block
  auto bar_p_ready = [&](int b) { return bar_base + 8u * (2 * SLOTS + 2 + b); };             // leader: weights in place
  auto bar_pv_done = [&](int b) { return bar_base + 8u * (2 * SLOTS + 4 + b); };             // both: O += P V finished
  const uint32_t bar_o_full = bar_base + 8u * (2 * SLOTS + 6), bar_q_ready = bar_base + 8u * (2 * SLOTS + 7);
  auto bar_s_free = [&](int b) { return bar_base + 8u * (2 * SLOTS + 8 + b); };              // leader: scores were read
  auto bar_m = [&](int grp, int q) { return bar_base + 8u * (2 * SLOTS + 10 + grp * 4 + q); };  // own: a row maximum was handed over
  auto bar_l = [&](int q) { return bar_base + 8u * (2 * SLOTS + 18 + q); };                     // own: both parts of the row sums

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  // One-dimensional grid in the order the CTAs should start: long tiles (late tokens of a causal call) first, and for
  // every tile (pair of neighbouring tiles) all KV heads before the next shorter one -- with the heads as a second grid
  // dimension the longest tiles of the last head would start last and set the launch's length.
  const int n_tiles = static_cast<int>(gridDim.x) / P.n_kv;        // even for pairs
  const int slot = static_cast<int>(blockIdx.x) / NCTA;            // cluster (or CTA) in start order
  const int kvh = slot % P.n_kv;
  const int tile = n_tiles - 1 - ((slot / P.n_kv) * NCTA + static_cast<int>(blockIdx.x) % NCTA);
  const int tok0 = tile * TOK;
  const int pair_tok0 = PAIR ? (tile & ~1) * TOK : tok0;           // tiles 2c and 2c + 1 share a cluster
  const unsigned long long tmo = P.timeout_ns;
  // An arrival of one warp on a barrier of the leading CTA.  Across the pair it is a relaxed arrive: what it announces
  // (scores read out of tensor memory; weights or K/V pieces written to this CTA's own shared memory) has been
  // completed and fenced for the tensor cores' proxy by the announcing threads before they get here, and a
  // cluster-scope release would make the warp wait for every outstanding memory operation of a busy SM.
  auto arrive_lead = [&](uint32_t bar) {
    if (!PAIR || rank == 0) mbar_arrive(bar);
    else mbar_arrive_cluster(map_to_cta(bar, 0));
  };

  if (tid == 0) {
    for (int s = 0; s < SLOTS; ++s) {
      mbar_init(bar_full(0, s), 4 * NCTA);  // one arrival per loader warp of the pair
      mbar_init(bar_empty(0, s), 1);        // the MMA commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_s_full(b), 1);          // the MMA commit
      mbar_init(bar_p_ready(b), 4 * NCTA);  // one arrival per softmax warp of the group, in both CTAs
      mbar_init(bar_pv_done(b), 1);
      mbar_init(bar_s_free(b), 4 * NCTA);   // the same
    }
    for (int q = 0; q < 4; ++q) {
      mbar_init(bar_m(0, q), 1);  // the warp of the group that owns these 32 rows
      mbar_init(bar_m(1, q), 1);
      mbar_init(bar_l(q), 2);     // that warp of either group
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_q_ready, 8 * NCTA);
    fence_mbar_init();
    s_abort_i = 0;
    s_lo = INT_MAX;
    s_hi = -1;
  }
  if (warp == 8) {
    if constexpr (PAIR) {
      tmem_alloc_pair(smem_u32(&s_tmem), Cfg::COLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&s_tmem), Cfg::COLS);
      tmem_relinquish();
    }
  }
  __syncthreads();
  // ---- key positions the pair needs: from the smallest first-visible to the largest last-visible of its tokens
  if (tid < NCTA * TOK && pair_tok0 + tid < P.n_rows) {
    const int qp = P.q_pos[pair_tok0 + tid];
    int lo = P.window > 0 ? qp - P.window + 1 : 0;
    lo = lo < P.seg_lo ? P.seg_lo : lo;
    const int hi = qp < P.seg_hi ? qp : P.seg_hi;
    if (hi >= lo) {
      atomicMin(&s_lo, lo);
      atomicMax(&s_hi, hi);
    }
  }
  tc_fence_before();
  if constexpr (PAIR) cluster_sync_all();  // barriers of both CTAs are initialised before anyone signals across the pair
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  const int blk0 = s_hi >= 0 ? s_lo / PT_KEYS : 0;
  const int n_blk = s_hi >= 0 ? s_hi / PT_KEYS - blk0 + 1 : 0;

  if (warp < 8) {
    // ------------------------------------------------------------------ softmax and epilogue: thread = MMA row
    // two warpgroups share the 128 rows: group 0 takes the even blocks, group 1 the odd ones, each with its own score
    // and weight buffer.  What a row carries from block to block is its running maximum, handed from group to group
    // through shared memory; every group keeps its own part of the row sum.
    const int wg = warp >> 2, q4 = warp & 3;
    const int row = q4 * 32 + lane;
    const int tok = tok0 + row / G, g = row % G;
    const bool valid = row / G < TOK && tok < P.n_rows;
    const int qp = valid ? P.q_pos[tok] : -1;
    const int lo = P.window > 0 ? qp - P.window + 1 : 0;
    const uint32_t lane_field = static_cast<uint32_t>(q4 * 32) << 16;
    const size_t row_off = (static_cast<size_t>(valid ? tok : 0) * P.n_q + kvh * G + (valid ? g : 0)) * D_HEAD;
    if (n_blk > 0) {
      // the query row into tensor memory: element pairs (2c, 2c + 1) -> column c (zeros for padding rows)
      const uint4 *qsrc = reinterpret_cast<const uint4 *>(P.q + row_off);
#pragma unroll 1
      for (int c = wg; c < D_HEAD / 64; c += 2) {
        uint32_t r[32];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 w = valid ? __ldg(qsrc + c * 8 + i) : make_uint4(0u, 0u, 0u, 0u);
          r[4 * i] = w.x;
          r[4 * i + 1] = w.y;
          r[4 * i + 2] = w.z;
          r[4 * i + 3] = w.w;
        }
        tmem_st_x32(tmem_base + lane_field + Cfg::COL_Q + c * 32, r);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) arrive_lead(bar_q_ready);
    }
    float m_own = -CUDART_INF_F;    // the maximum this group's part of the row sum refers to
    uint64_t l2[2] = {0ull, 0ull};  // that part, in four chains (two packed pairs)
    bool ok = true;
    const uint64_t c2 = pack2(P.scale_log2e, P.scale_log2e), one2 = pack2(1.0f, 1.0f);
    const int buf = wg;
    for (int j = wg; j < n_blk; j += 2) {
      const uint32_t ph = (j >> 1) & 1;
      if (!polite_warp_wait(bar_s_full(buf), ph, s_abort, tmo, lane)) {
        raise(P.status, STATUS_TIMEOUT, s_abort);
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t s_col = tmem_base + lane_field + Cfg::COL_S + buf * PT_KEYS;
      uint32_t s0[32], s1[32];
      tmem_ld_x32(s_col, s0);
      tmem_ld_x32(s_col + 32, s1);
      // which keys of the block does this row see: present in a segment, not after the row's position, inside its window
      const int pos0 = (blk0 + j) * PT_KEYS;
      unsigned long long vis = 0ull;
#pragma unroll
      for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
        int a = P.first[sg] - pos0, b = P.first[sg] + P.len[sg] - pos0;  // [a, b) of the block's key slots
        a = a < 0 ? 0 : a;
        b = b > PT_KEYS ? PT_KEYS : b;
        if (b > a) vis |= (b - a == 64 ? ~0ull : ((1ull << (b - a)) - 1ull) << a);
      }
      {
        int a = lo - pos0, b = qp - pos0 + 1;
        a = a < 0 ? 0 : a;
        b = b > PT_KEYS ? PT_KEYS : b;
        vis &= b > a ? (b - a == 64 ? ~0ull : ((1ull << (b - a)) - 1ull) << a) : 0ull;
      }
      tmem_wait_ld();
      // the scores are in registers: their columns may take this group's next block
      tc_fence_before();
      __syncwarp();
      if (lane == 0) arrive_lead(bar_s_free(buf));
      if (!__all_sync(0xffffffffu, vis == ~0ull)) {
        const uint32_t v0 = static_cast<uint32_t>(vis), v1 = static_cast<uint32_t>(vis >> 32);
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          if (!((v0 >> k) & 1u)) s0[k] = 0xff800000u;  // -inf
          if (!((v1 >> k) & 1u)) s1[k] = 0xff800000u;
        }
      }
      // the block's maximum in four chains of three-input maxima
      float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int k = 0; k < 32; k += 8) {
        mx[0] = fmax3(mx[0], __uint_as_float(s0[k]), __uint_as_float(s0[k + 1]));
        mx[1] = fmax3(mx[1], __uint_as_float(s0[k + 2]), __uint_as_float(s0[k + 3]));
        mx[2] = fmax3(mx[2], __uint_as_float(s0[k + 4]), __uint_as_float(s0[k + 5]));
        mx[3] = fmax3(mx[3], __uint_as_float(s0[k + 6]), __uint_as_float(s0[k + 7]));
        mx[0] = fmax3(mx[0], __uint_as_float(s1[k]), __uint_as_float(s1[k + 1]));
        mx[1] = fmax3(mx[1], __uint_as_float(s1[k + 2]), __uint_as_float(s1[k + 3]));
        mx[2] = fmax3(mx[2], __uint_as_float(s1[k + 4]), __uint_as_float(s1[k + 5]));
        mx[3] = fmax3(mx[3], __uint_as_float(s1[k + 6]), __uint_as_float(s1[k + 7]));
      }
      const float bm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * P.scale_log2e;  // log2 units (scale > 0)
      // the row's maximum after block j - 1 comes from the other group; the one after block j goes back to it
      float m_prev = -CUDART_INF_F;
      if (j > 0) {
        if (!polite_warp_wait(bar_m(wg ^ 1, q4), ((j - 1) >> 1) & 1, s_abort, tmo, lane)) {
          raise(P.status, STATUS_TIMEOUT, s_abort);
          ok = false;
          break;
        }
        m_prev = s_mx[wg ^ 1][row];
      }
      // The reference m the weights 2^(s - m) are taken against follows the row's maximum lazily: it moves (and O and
      // the row sums are rescaled) only when a block's maximum exceeds it by more than 2^PT_TAU; until then the
      // weights may reach 2^PT_TAU, which fp32 sums and 16-bit weights hold as well as values below 1.  A function of
      // the row's own scores and of the block order alone, like the maximum itself.
      const float m_new = m_prev == -CUDART_INF_F ? bm : (bm > m_prev + PT_TAU ? bm : m_prev);
      s_mx[wg][row] = m_new;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_m(wg, q4));
      const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
      // rescale of what the row has so far: exactly 1 when its maximum stays; while nothing has been seen O and l are 0
      const float alpha = m_prev == -CUDART_INF_F ? 1.0f : ex2_approx(m_prev - m_use);
      const float alpha_own = m_own == -CUDART_INF_F ? 1.0f : ex2_approx(m_own - m_use);
      m_own = m_new;
      // weights 2^(s * scale - m): two per fused multiply-add; the row sum adds them up in fp32, the product takes
      // them rounded to the element type
      uint32_t w[32];
      const uint64_t nm2 = pack2(-m_use, -m_use), al2 = pack2(alpha_own, alpha_own);
      l2[0] = fmul2(l2[0], al2);
      l2[1] = fmul2(l2[1], al2);
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        float e0, e1;
        unpack2(ffma2(pack2(__uint_as_float(s0[k]), __uint_as_float(s0[k + 1])), c2, nm2), e0, e1);
        const float p0 = ex2_approx(e0), p1 = ex2_approx(e1);
        w[k >> 1] = pack_out<DT>(p0, p1);
        l2[(k >> 1) & 1] = ffma2(pack2(p0, p1), one2, l2[(k >> 1) & 1]);
      }
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        float e0, e1;
        unpack2(ffma2(pack2(__uint_as_float(s1[k]), __uint_as_float(s1[k + 1])), c2, nm2), e0, e1);
        const float p0 = ex2_approx(e0), p1 = ex2_approx(e1);
        w[16 + (k >> 1)] = pack_out<DT>(p0, p1);
        l2[(k >> 1) & 1] = ffma2(pack2(p0, p1), one2, l2[(k >> 1) & 1]);
      }
      // P_j into shared memory as a K-major A operand (row = MMA row, 128 bytes = 64 keys, 128-byte swizzle); the
      // product that read this buffer two blocks ago has long finished
      if (j >= 2 && !polite_warp_wait(bar_pv_done(buf), ((j - 2) >> 1) & 1, s_abort, tmo, lane)) {
        raise(P.status, STATUS_TIMEOUT, s_abort);
        ok = false;
        break;
      }
      if constexpr (Cfg::P_TMEM) {
        tmem_st_x32(tmem_base + lane_field + Cfg::COL_P + buf * (PT_KEYS / 2), w);
      } else {
        const uint32_t prow = p_smem + buf * Cfg::P_BYTES + row * 128;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(prow + ((i ^ (row & 7)) << 4)), "r"(w[4 * i]), "r"(w[4 * i + 1]),
                       "r"(w[4 * i + 2]), "r"(w[4 * i + 3])
                       : "memory");
        fence_proxy_async_smem();
      }
      if (__any_sync(0xffffffffu, alpha != 1.0f)) {
        // O holds the blocks before j; the last of those products must have finished (j >= 1 here: a maximum exists)
        if (!polite_warp_wait(bar_pv_done(buf ^ 1), ((j - 1) >> 1) & 1, s_abort, tmo, lane)) {
          raise(P.status, STATUS_TIMEOUT, s_abort);
          ok = false;
          break;
        }
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < D_HEAD / 32; ++c) {
          uint32_t r[32];
          tmem_ld_x32(tmem_base + lane_field + Cfg::COL_O + c * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
          tmem_st_x32(tmem_base + lane_field + Cfg::COL_O + c * 32, r);
        }
        tmem_wait_st();
        tc_fence_before();
      } else if constexpr (Cfg::P_TMEM) {
        tmem_wait_st();
        tc_fence_before();
      }
      __syncwarp();
      if (lane == 0) arrive_lead(bar_p_ready(buf));
    }
    // ---- the row sum: both parts referred to the final maximum, added in group order
    float l_run = 0.f;
    if (ok && n_blk > 0) {
      const int last = n_blk - 1;
      float m_fin = m_own;
      if ((last & 1) != wg) {
        if (!polite_warp_wait(bar_m(wg ^ 1, q4), (last >> 1) & 1, s_abort, tmo, lane)) {
          raise(P.status, STATUS_TIMEOUT, s_abort);
          ok = false;
        }
        m_fin = s_mx[wg ^ 1][row];
      }
      if (ok) {
        const float m_use = m_fin == -CUDART_INF_F ? 0.f : m_fin;
        float a0, a1, a2, a3;
        unpack2(l2[0], a0, a1);
        unpack2(l2[1], a2, a3);
        const float mine = ((a0 + a1) + (a2 + a3)) * (m_own == -CUDART_INF_F ? 1.0f : ex2_approx(m_own - m_use));
        s_lx[wg][row] = mine;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_l(q4));
        if (!polite_warp_wait(bar_l(q4), 0, s_abort, tmo, lane)) {
          raise(P.status, STATUS_TIMEOUT, s_abort);
          ok = false;
        }
        l_run = s_lx[0][row] + s_lx[1][row];
      }
    }
    // ---- normalise and store, each group its half of the channels (a token without a visible key yields zeros)
    if (ok && n_blk > 0 && !polite_warp_wait(bar_o_full, 0, s_abort, tmo, lane)) {
      raise(P.status, STATUS_TIMEOUT, s_abort);
      ok = false;
    }
    if (ok) {
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
      uint4 *dst = reinterpret_cast<uint4 *>(P.out + row_off);
#pragma unroll 1
      for (int c = wg * (D_HEAD / 64); c < (wg + 1) * (D_HEAD / 64); ++c) {
        uint32_t r[32];
        if (n_blk > 0) {
          tmem_ld_x32(tmem_base + lane_field + Cfg::COL_O + c * 32, r);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
        uint32_t o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = pack_out<DT>(__uint_as_float(r[2 * i]) * inv, __uint_as_float(r[2 * i + 1]) * inv);
        if (valid) {
#pragma unroll
          for (int i = 0; i < 4; ++i) dst[c * 4 + i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        }
      }
    }
  } else if (warp == 8 || warp == 9) {
    // ------------------------------------------------------------------ MMA issue (one thread per product, leading CTA)
    constexpr uint32_t IDESC_BASE = (DT == 0 ? umma_idesc_bf16_f32(PT_ROWS * NCTA, 8) : umma_idesc_f16_f32(PT_ROWS * NCTA, 8)) & ~(1u << 17);
    constexpr uint32_t IDESC_S = IDESC_BASE | (static_cast<uint32_t>(PT_KEYS >> 3) << 17);              // N = 64 keys, B K-major
    constexpr uint32_t IDESC_O = IDESC_BASE | (static_cast<uint32_t>(D_HEAD >> 3) << 17) | (1u << 16);  // N = d_head, B MN-major
    auto commit = [&](uint32_t bar) {
      if constexpr (PAIR) umma_commit_pair(bar, 3);  // the barrier at this offset in both CTAs
      else umma_commit(bar);
    };
    if (lane == 0 && n_blk > 0 && rank == 0 && warp == 8) {
      // S_j = Q K_j^T into score buffer j & 1, as far ahead of the softmax as the two buffers allow
      bool ok = lead_wait<PAIR>(bar_q_ready, 0, s_abort, tmo);
      tc_fence_after();
      for (int j = 0; ok && j < n_blk; ++j) {
        const int slot = j % SLOTS_K;
        // the K block has landed; the softmax threads have read the scores of block j - 2 out of these columns
        if (!lead_wait<PAIR>(bar_full(0, slot), (j / SLOTS_K) & 1, s_abort, tmo) ||
            (j >= 2 && !lead_wait<PAIR>(bar_s_free(j & 1), ((j - 2) >> 1) & 1, s_abort, tmo))) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d = tmem_base + Cfg::COL_S + (j & 1) * PT_KEYS;
        const uint64_t desc0 = umma_smem_desc_sw128(ring + slot * Cfg::TILE_BYTES);
#pragma unroll
        for (int ks = 0; ks < D_HEAD / 16; ++ks) {
          const uint64_t bdesc = desc0 + (((ks >> 2) * Cfg::SLAB_K + (ks & 3) * 32) >> 4);
          if constexpr (PAIR) umma_f16_ts_pair(d, tmem_base + Cfg::COL_Q + ks * 8, bdesc, IDESC_S, ks > 0 ? 1u : 0u);
          else umma_f16_ts(d, tmem_base + Cfg::COL_Q + ks * 8, bdesc, IDESC_S, ks > 0 ? 1u : 0u);
        }
        commit(bar_empty(0, slot));
        commit(bar_s_full(j & 1));
      }
      if (!ok) raise(P.status, STATUS_TIMEOUT, s_abort);
    } else if (lane == 0 && n_blk > 0 && rank == 0) {
      // O += P_j V_j once the weights are in place (and O has been rescaled where a reference maximum moved)
      bool ok = true;
      for (int j = 0; j < n_blk; ++j) {
        const int slot = j % SLOTS_V;
        if (!lead_wait<PAIR>(bar_p_ready(j & 1), (j >> 1) & 1, s_abort, tmo) ||
            !lead_wait<PAIR>(bar_full(1, slot), (j / SLOTS_V) & 1, s_abort, tmo)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint64_t desc0 = umma_smem_desc_sw128_mn(ring_v + slot * Cfg::TILE_BYTES, Cfg::SLAB_V);
        const uint64_t pdesc0 = umma_smem_desc_sw128(p_smem + (j & 1) * Cfg::P_BYTES);
        const uint32_t ptmem = tmem_base + Cfg::COL_P + (j & 1) * (PT_KEYS / 2);
#pragma unroll
        for (int ks = 0; ks < PT_KEYS / 16; ++ks) {
          const uint64_t vdesc = desc0 + ((ks * 16 * 128) >> 4);
          const uint32_t acc = (j > 0 || ks > 0) ? 1u : 0u;
          if constexpr (Cfg::P_TMEM) {
            if constexpr (PAIR) umma_f16_ts_pair(tmem_base + Cfg::COL_O, ptmem + ks * 8, vdesc, IDESC_O, acc);
            else umma_f16_ts(tmem_base + Cfg::COL_O, ptmem + ks * 8, vdesc, IDESC_O, acc);
          } else {
            if constexpr (PAIR) umma_bf16_pair(tmem_base + Cfg::COL_O, pdesc0 + ((ks * 32) >> 4), vdesc, IDESC_O, acc);
            else umma_bf16(tmem_base + Cfg::COL_O, pdesc0 + ((ks * 32) >> 4), vdesc, IDESC_O, acc);
          }
        }
        commit(bar_empty(1, slot));
        commit(bar_pv_done(j & 1));
      }
      if (ok) commit(bar_o_full);
      else raise(P.status, STATUS_TIMEOUT, s_abort);
    }
  } else {
    // ------------------------------------------------------------------ K/V blocks into the rings
    // issue order = the order the products want them, the keys three blocks ahead: K_0 K_1 K_2 | K_3 V_0 | K_4 V_1 | ...
    // This CTA's share of a block: K_ROWS keys of all channels (K), all 64 keys of V_COLS channels (V).
    const int ptid = tid - 10 * 32;
    // blocks issued and not yet published to the MMA threads, oldest first.  A block is published once PT_LAG younger
    // ones have been issued -- or at once, all of them, when the next block would have to wait for a free slot (the
    // slot is freed by a product that may itself be waiting for one of these blocks).
    uint32_t pend[PT_LAG + 1] = {};
    int n_pend = 0;
    bool ok = true;
    auto publish_all = [&]() {
      cp_async_wait_all();
      fence_proxy_async_smem();
      __syncwarp();
#pragma unroll
      for (int i = 0; i <= PT_LAG; ++i)
        if (i < n_pend && lane == 0) arrive_lead(pend[i]);
      n_pend = 0;
    };
    // rows [row_first, row_first + ROWS) of the block, CPR 16-byte pieces of each starting at element col_first
    auto gather = [&](auto rows_c, auto cpr_c, uint32_t base, int slab_bytes, int pos_first, int col_first, bool is_v) {
      constexpr int ROWS = decltype(rows_c)::value, CPR = decltype(cpr_c)::value;
      constexpr int RSTEP = PT_LOADERS / CPR;  // rows one pass of the 128 threads covers
      const int c = ptid % CPR, r0 = ptid / CPR;
      const uint32_t dst = base + static_cast<uint32_t>(c >> 3) * slab_bytes;
      // the usual case: one segment holds all the rows -> one base pointer, one stride
      int whole = -1;
#pragma unroll
      for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg)
        if (P.first[sg] <= pos_first && pos_first + ROWS <= P.first[sg] + P.len[sg]) whole = sg;
      if (whole >= 0) {
        const long long stride = P.stride[whole];
        const __nv_bfloat16 *src = (is_v ? P.v[whole] : P.k[whole]) + static_cast<size_t>(pos_first - P.first[whole] + r0) * stride +
                                   static_cast<size_t>(kvh) * D_HEAD + col_first + c * 8;
#pragma unroll
        for (int pass = 0; pass < ROWS / RSTEP; ++pass) {
          const int r = r0 + pass * RSTEP;
          cp_async16(dst + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, true);
          src += RSTEP * stride;
        }
      } else {
#pragma unroll 1
        for (int pass = 0; pass < ROWS / RSTEP; ++pass) {
          const int r = r0 + pass * RSTEP, pos = pos_first + r;
          const __nv_bfloat16 *src = P.q;
          bool have = false;
#pragma unroll
          for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
            const int rr = pos - P.first[sg];
            if (rr >= 0 && rr < P.len[sg]) {
              src = (is_v ? P.v[sg] : P.k[sg]) + static_cast<size_t>(rr) * P.stride[sg] + static_cast<size_t>(kvh) * D_HEAD + col_first + c * 8;
              have = true;
            }
          }
          cp_async16(dst + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, have);
        }
      }
    };
    auto emit = [&](int is_v, int j) -> bool {
      const int n_slots = is_v ? SLOTS_V : SLOTS_K, slot = j % n_slots;
      if (j >= n_slots) {
        const uint32_t par = ((j / n_slots) - 1) & 1;
        int free_now = lane == 0 ? (mbar_try_wait(bar_empty(is_v, slot), par) ? 1 : 0) : 0;
        free_now = __shfl_sync(0xffffffffu, free_now, 0);
        if (!free_now) {
          publish_all();
          int got = lane == 0 ? (polite_wait<false>(bar_empty(is_v, slot), par, s_abort, tmo) ? 1 : 0) : 0;
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) return false;
        }
      }
      const int pos0 = (blk0 + j) * PT_KEYS;
      if (is_v)
        gather(std::integral_constant<int, PT_KEYS>(), std::integral_constant<int, Cfg::V_COLS / 8>(), ring_v + slot * Cfg::TILE_BYTES,
               Cfg::SLAB_V, pos0, static_cast<int>(rank) * Cfg::V_COLS, true);
      else
        gather(std::integral_constant<int, Cfg::K_ROWS>(), std::integral_constant<int, D_HEAD / 8>(), ring + slot * Cfg::TILE_BYTES,
               Cfg::SLAB_K, pos0 + static_cast<int>(rank) * Cfg::K_ROWS, 0, false);
      cp_async_commit();
#pragma unroll
      for (int i = 0; i <= PT_LAG; ++i)
        if (i == n_pend) pend[i] = bar_full(is_v, slot);
      ++n_pend;
      if (n_pend > PT_LAG) {
        // the oldest block has PT_LAG younger ones behind it: it has landed by now, or nearly
        cp_async_wait_group<PT_LAG>();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) arrive_lead(pend[0]);
#pragma unroll
        for (int i = 0; i < PT_LAG; ++i) pend[i] = pend[i + 1];
        --n_pend;
      }
      return true;
    };
    if (n_blk > 0) {
      ok = emit(0, 0);
      if (ok && n_blk > 1) ok = emit(0, 1);
      if (ok && n_blk > 2) ok = emit(0, 2);
      for (int j = 0; ok && j < n_blk; ++j) {
        if (j + 3 < n_blk) ok = emit(0, j + 3);
        if (ok) ok = emit(1, j);
      }
      if (ok) publish_all();
      else {
        cp_async_wait_all();
        raise(P.status, STATUS_TIMEOUT, s_abort);
      }
    }
  }

  // ---- teardown: every role is done with tensor memory; in a pair nobody leaves while the partner can still signal
  // into this CTA's shared memory
  tc_fence_before();
  if constexpr (PAIR) cluster_sync_all();
  else __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    if constexpr (PAIR) tmem_dealloc_pair(tmem_base, Cfg::COLS);
    else tmem_dealloc(tmem_base, Cfg::COLS);
  }
}

template <int D_HEAD, int G, bool PAIR>
static kvd_status prefill_tc_launch(kvd_ctx *ctx, const PrefillParams &P, cudaStream_t stream) {
  using Cfg = PtCfg<D_HEAD, PAIR>;
  auto k0 = kvd_prefill_attn_tc_kernel<D_HEAD, G, 0, PAIR>;
  auto k1 = kvd_prefill_attn_tc_kernel<D_HEAD, G, 1, PAIR>;
  static bool configured[64] = {};
  if (!configured[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(k0, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(prefill attention)");
    configured[ctx->device & 63] = true;
  }
  const int tok = PT_ROWS / G;
  int tiles = (P.n_rows + tok - 1) / tok;
  if (PAIR) tiles = (tiles + 1) & ~1;  // whole pairs: a CTA whose tile lies past the last row has no rows to store
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(tiles * P.n_kv, 1, 1);
  cfg.blockDim = dim3(PT_THREADS, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = ctx->dtype == 1 ? cudaLaunchKernelEx(&cfg, k1, P) : cudaLaunchKernelEx(&cfg, k0, P);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prefill attention");
  ctx->launches += 1;
  return KVD_OK;
}

template <int D_HEAD>
static kvd_status prefill_tc_group(kvd_ctx *ctx, const PrefillParams &P, int group, cudaStream_t stream) {
  // pairs where the K/V bytes per block bound the kernel (d_head = 256); at 128 the softmax does, and the hand-overs
  // across the pair cost more than the halved traffic returns (measured).  KVD_PREFILL_PAIR=0/1 overrides, for comparisons.
  static const char *env = getenv("KVD_PREFILL_PAIR");
  const bool pair = D_HEAD >= 128 && (env ? env[0] == '1' : D_HEAD == 256);
  if constexpr (D_HEAD >= 128) {
    if (pair) {
      switch (group) {
        case 1: return prefill_tc_launch<D_HEAD, 1, true>(ctx, P, stream);
        case 2: return prefill_tc_launch<D_HEAD, 2, true>(ctx, P, stream);
        case 3: return prefill_tc_launch<D_HEAD, 3, true>(ctx, P, stream);
        case 4: return prefill_tc_launch<D_HEAD, 4, true>(ctx, P, stream);
        case 8: return prefill_tc_launch<D_HEAD, 8, true>(ctx, P, stream);
        default: return KVD_ERR_SHAPE;
      }
    }
  }
  switch (group) {
    case 1: return prefill_tc_launch<D_HEAD, 1, false>(ctx, P, stream);
    case 2: return prefill_tc_launch<D_HEAD, 2, false>(ctx, P, stream);
    case 3: return prefill_tc_launch<D_HEAD, 3, false>(ctx, P, stream);
    case 4: return prefill_tc_launch<D_HEAD, 4, false>(ctx, P, stream);
    case 8: return prefill_tc_launch<D_HEAD, 8, false>(ctx, P, stream);
    default: return KVD_ERR_SHAPE;
  }
}

kvd_status launch_prefill_tc(kvd_ctx *ctx, const PrefillParams &P, int d_head, int group, cudaStream_t stream) {
  switch (d_head) {
    case 64: return prefill_tc_group<64>(ctx, P, group, stream);
    case 128: return prefill_tc_group<128>(ctx, P, group, stream);
    case 256: return prefill_tc_group<256>(ctx, P, group, stream);
    default: return KVD_ERR_SHAPE;
  }
}

}  // namespace kvd
