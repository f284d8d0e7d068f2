// ATTENTION of Algorithm 1 (Eq. 6-7) for many query tokens of one sequence on the fifth-generation tensor cores.
//
//   CTA   = (tile of query tokens, KV head): 128 MMA rows = 128 / Gp tokens x Gp query heads of the head's group
//           (Gp = group size rounded up to a power of two; padding heads are zero rows that are never stored).
//   keys  = blocks of 64, aligned to ABSOLUTE position, walked in ascending order from the first block any row of the
//           tile can see to the last one.
//   TMEM  = [ O : d_head columns | S_0, S_1 : 64 columns each | Q : d_head / 2 columns ].  The query tile is written
//           there once (two elements per 32-bit column) and is the A operand of S_j = Q K_j^T; the softmax threads
//           read S_j (one row per thread, no shuffles), write the weights P_j over it in the element type, and P_j is
//           the A operand of O += P_j V_j.  Both products are tcgen05.mma with A from tensor memory; shared memory
//           holds nothing but a ring of K and V blocks.
//   warps = 0-3 softmax and epilogue (TMEM lane quarter = warp), 4 issues the MMAs, 5-8 gather K/V blocks from the
//           segments with 16-byte cp.async into the 128-byte-swizzled layouts the two products expect (K block:
//           K-major B operand, rows = keys; V block: the same bytes read as an MN-major B operand, rows = the
//           contraction index).  Positions no segment holds are zero-filled and masked.
//   order = S_0 | S_1 PV_0 | S_2 PV_1 | ... : S_{j+1} runs on the tensor cores while the softmax of block j runs on
//           the ALUs; the two S buffers alternate.  The running maximum of a row changes rarely after its first blocks;
//           O is rescaled in tensor memory only when a row of the warp needs it (the others multiply by exactly 1).
//
// A row's result depends on that row alone: the rows of an MMA are computed independently, every row walks the key
// blocks of its tile in ascending order, a block without a visible key for the row changes nothing for it (weights 0,
// rescale by exactly 1, O += 0), and the block boundaries are absolute.  So a token attended alone and the same token
// inside any tile give the same bits.  They are not the bits of kvd_decode_attention (another split of the keys, P
// rounded before the second product).  Every wait is bounded: on a timeout the CTA raises the status word, all roles
// leave their loops, and tensor memory is freed.
#include <math_constants.h>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

constexpr int PT_ROWS = 128;     // MMA rows per CTA
constexpr int PT_KEYS = 64;      // keys per block
constexpr int PT_THREADS = 288;  // nine warps
constexpr int PT_LOADERS = 128;  // threads of warps 5-8
constexpr int PT_LAG = 3;        // blocks a loader thread keeps in flight behind the one it is issuing

template <int D_HEAD>
struct PtCfg {
  static constexpr int TILE_BYTES = PT_KEYS * D_HEAD * 2;       // one K or V block
  static constexpr int SLAB_BYTES = PT_KEYS * 128;              // 64 channels of every key of a block
  static constexpr int SLOTS = D_HEAD == 256 ? 6 : 8;           // ring of blocks
  static constexpr int COL_O = 0, COL_S = D_HEAD, COL_Q = D_HEAD + 2 * PT_KEYS;
  static constexpr int COLS_USED = COL_Q + D_HEAD / 2;
  static constexpr int COLS = COLS_USED <= 256 ? 256 : 512;     // allocation: a power of two
  static constexpr int N_BARS = 2 * SLOTS + 8;
  static constexpr int SMEM_BYTES = 1024 + SLOTS * TILE_BYTES + N_BARS * 8;
};

template <int D_HEAD, int G, int DT>
__global__ void __launch_bounds__(PT_THREADS, 1) kvd_prefill_attn_tc_kernel(const __grid_constant__ PrefillParams P) {
  using Cfg = PtCfg<D_HEAD>;
  constexpr int GP = G == 3 ? 4 : G;   // heads of the group, padded to a power of two
  constexpr int TOK = PT_ROWS / GP;    // query tokens per CTA
  constexpr int SLOTS = Cfg::SLOTS;
  extern __shared__ uint8_t pt_smem_raw[];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort_i, s_lo, s_hi;
  volatile int *s_abort = &s_abort_i;
  // the ring starts on a 1024-byte boundary (the swizzle is a function of the address), the barriers follow it
  const uint32_t ring = (smem_u32(pt_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = ring + SLOTS * Cfg::TILE_BYTES;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty = [&](int s) { return bar_base + 8u * (SLOTS + s); };
  auto bar_s_full = [&](int b) { return bar_base + 8u * (2 * SLOTS + b); };
  auto bar_p_ready = [&](int b) { return bar_base + 8u * (2 * SLOTS + 2 + b); };
  auto bar_pv_done = [&](int b) { return bar_base + 8u * (2 * SLOTS + 4 + b); };
  const uint32_t bar_o_full = bar_base + 8u * (2 * SLOTS + 6), bar_q_ready = bar_base + 8u * (2 * SLOTS + 7);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // long tiles (late tokens of a causal call) first
  const int tok0 = (static_cast<int>(gridDim.x) - 1 - static_cast<int>(blockIdx.x)) * TOK, kvh = blockIdx.y;
  const unsigned long long tmo = P.timeout_ns;

  if (tid == 0) {
    for (int s = 0; s < SLOTS; ++s) {
      mbar_init(bar_full(s), PT_LOADERS);  // one arrival per loader thread
      mbar_init(bar_empty(s), 1);          // the MMA commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_s_full(b), 1);         // the MMA commit
      mbar_init(bar_p_ready(b), PT_ROWS);  // one arrival per softmax thread
      mbar_init(bar_pv_done(b), 1);
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_q_ready, PT_ROWS);
    fence_mbar_init();
    s_abort_i = 0;
    s_lo = INT_MAX;
    s_hi = -1;
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&s_tmem), Cfg::COLS);
    tmem_relinquish();
  }
  __syncthreads();
  // ---- key positions the tile needs: from the smallest first-visible to the largest last-visible of its tokens
  if (tid < TOK && tok0 + tid < P.n_rows) {
    const int qp = P.q_pos[tok0 + tid];
    int lo = P.window > 0 ? qp - P.window + 1 : 0;
    lo = lo < P.seg_lo ? P.seg_lo : lo;
    const int hi = qp < P.seg_hi ? qp : P.seg_hi;
    if (hi >= lo) {
      atomicMin(&s_lo, lo);
      atomicMax(&s_hi, hi);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  const int blk0 = s_hi >= 0 ? s_lo / PT_KEYS : 0;
  const int n_blk = s_hi >= 0 ? s_hi / PT_KEYS - blk0 + 1 : 0;

  if (warp < 4) {
    // ------------------------------------------------------------------ softmax and epilogue: thread = MMA row
    const int row = tid;
    const int tok = tok0 + row / GP, g = row % GP;
    const bool valid = tok < P.n_rows && g < G;
    const int qp = valid ? P.q_pos[tok] : -1;
    const int lo = P.window > 0 ? qp - P.window + 1 : 0;
    const uint32_t lane_field = static_cast<uint32_t>(warp * 32) << 16;
    const size_t row_off = (static_cast<size_t>(valid ? tok : 0) * P.n_q + kvh * G + (valid ? g : 0)) * D_HEAD;
    if (n_blk > 0) {
      // the query row into tensor memory: element pairs (2c, 2c + 1) -> column c (zeros for padding rows)
      const uint4 *qsrc = reinterpret_cast<const uint4 *>(P.q + row_off);
#pragma unroll 1
      for (int c = 0; c < D_HEAD / 64; ++c) {
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
      mbar_arrive(bar_q_ready);
    }
    float m_run = -CUDART_INF_F, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_blk; ++j) {
      const int buf = j & 1;
      if (!warp_wait(bar_s_full(buf), (j >> 1) & 1, s_abort, tmo, lane)) {
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
      if (!__all_sync(0xffffffffu, vis == ~0ull)) {
        const uint32_t v0 = static_cast<uint32_t>(vis), v1 = static_cast<uint32_t>(vis >> 32);
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          if (!((v0 >> k) & 1u)) s0[k] = 0xff800000u;  // -inf
          if (!((v1 >> k) & 1u)) s1[k] = 0xff800000u;
        }
      }
      // the block's maximum in four chains
      float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        mx[k & 3] = fmaxf(mx[k & 3], __uint_as_float(s0[k]));
        mx[k & 3] = fmaxf(mx[k & 3], __uint_as_float(s1[k]));
      }
      const float bm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * P.scale_log2e;  // log2 units (scale > 0)
      const float m_new = fmaxf(m_run, bm);
      const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
      // rescale of what the row has so far: exactly 1 when its maximum stays; while nothing has been seen O and l are 0
      const float alpha = m_run == -CUDART_INF_F ? 1.0f : ex2_approx(m_run - m_use);
      m_run = m_new;
      // weights, rounded to the element type (the rounded weights are also what the row sum adds up)
      uint32_t w[32];
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(s0[k]), P.scale_log2e, -m_use));
        const float p1 = ex2_approx(fmaf(__uint_as_float(s0[k + 1]), P.scale_log2e, -m_use));
        w[k >> 1] = pack_out<DT>(p0, p1);
        float r0, r1;
        unpack2(x2_to_f32x2<DT>(w[k >> 1]), r0, r1);
        ls[(k >> 1) & 3] += r0 + r1;
      }
#pragma unroll
      for (int k = 0; k < 32; k += 2) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(s1[k]), P.scale_log2e, -m_use));
        const float p1 = ex2_approx(fmaf(__uint_as_float(s1[k + 1]), P.scale_log2e, -m_use));
        w[16 + (k >> 1)] = pack_out<DT>(p0, p1);
        float r0, r1;
        unpack2(x2_to_f32x2<DT>(w[16 + (k >> 1)]), r0, r1);
        ls[(k >> 1) & 3] += r0 + r1;
      }
      l_run = fmaf(l_run, alpha, (ls[0] + ls[1]) + (ls[2] + ls[3]));
      tmem_st_x32(s_col, w);  // P_j over the first half of S_j
      if (__any_sync(0xffffffffu, alpha != 1.0f)) {
        // O holds the blocks before j; the last of those products must have finished (j >= 1 here: a maximum exists)
        if (!warp_wait(bar_pv_done((j - 1) & 1), ((j - 1) >> 1) & 1, s_abort, tmo, lane)) {
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
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p_ready(buf));
    }
    // ---- normalise and store (a token without a visible key yields zeros)
    if (ok && n_blk > 0 && !warp_wait(bar_o_full, 0, s_abort, tmo, lane)) {
      raise(P.status, STATUS_TIMEOUT, s_abort);
      ok = false;
    }
    if (ok) {
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
      uint4 *dst = reinterpret_cast<uint4 *>(P.out + row_off);
#pragma unroll 1
      for (int c = 0; c < D_HEAD / 32; ++c) {
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
  } else if (warp == 4) {
    // ------------------------------------------------------------------ MMA issue (one thread)
    if (lane == 0 && n_blk > 0) {
      constexpr uint32_t IDESC_BASE = DT == 0 ? umma_idesc_bf16_f32(PT_ROWS, 8) & ~(1u << 17) : umma_idesc_f16_f32(PT_ROWS, 8) & ~(1u << 17);
      constexpr uint32_t IDESC_S = IDESC_BASE | (static_cast<uint32_t>(PT_KEYS >> 3) << 17);                 // N = 64 keys, B K-major
      constexpr uint32_t IDESC_O = IDESC_BASE | (static_cast<uint32_t>(D_HEAD >> 3) << 17) | (1u << 16);     // N = d_head, B MN-major
      int t = 0;  // blocks taken from the ring so far
      bool ok = mbar_wait(bar_q_ready, 0, s_abort, tmo);
      if (!ok) raise(P.status, STATUS_TIMEOUT, s_abort);
      tc_fence_after();
      // S_j = Q K_j^T into score buffer j & 1
      auto issue_s = [&](int j) -> bool {
        const int slot = t % SLOTS;
        if (!mbar_wait(bar_full(slot), (t / SLOTS) & 1, s_abort, tmo)) return false;
        tc_fence_after();
        const uint32_t kb = ring + slot * Cfg::TILE_BYTES;
        const uint32_t d = tmem_base + Cfg::COL_S + (j & 1) * PT_KEYS;
#pragma unroll
        for (int ks = 0; ks < D_HEAD / 16; ++ks)
          umma_f16_ts(d, tmem_base + Cfg::COL_Q + ks * 8, umma_smem_desc_sw128(kb + (ks >> 2) * Cfg::SLAB_BYTES + (ks & 3) * 32),
                      IDESC_S, ks > 0 ? 1u : 0u);
        umma_commit(bar_empty(slot));
        umma_commit(bar_s_full(j & 1));
        ++t;
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int j = 0; ok && j < n_blk; ++j) {
        if (j + 1 < n_blk && !issue_s(j + 1)) {
          ok = false;
          break;
        }
        // O += P_j V_j once the weights are in place (and O has been rescaled where a maximum moved)
        const int slot = t % SLOTS;
        if (!mbar_wait(bar_p_ready(j & 1), (j >> 1) & 1, s_abort, tmo) || !mbar_wait(bar_full(slot), (t / SLOTS) & 1, s_abort, tmo)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t vb = ring + slot * Cfg::TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < PT_KEYS / 16; ++ks)
          umma_f16_ts(tmem_base + Cfg::COL_O, tmem_base + Cfg::COL_S + (j & 1) * PT_KEYS + ks * 8,
                      umma_smem_desc_sw128_mn(vb + ks * 16 * 128, Cfg::SLAB_BYTES), IDESC_O, (j > 0 || ks > 0) ? 1u : 0u);
        umma_commit(bar_empty(slot));
        umma_commit(bar_pv_done(j & 1));
        ++t;
      }
      if (ok) umma_commit(bar_o_full);
      else raise(P.status, STATUS_TIMEOUT, s_abort);
    }
  } else {
    // ------------------------------------------------------------------ K/V blocks into the ring
    // ring order = the order the MMA thread consumes them: K_0 | K_1 V_0 | K_2 V_1 | ...
    constexpr int CPR = D_HEAD / 8;           // 16-byte pieces per key
    constexpr int RSTEP = PT_LOADERS / CPR;   // keys one pass of the 128 threads covers
    const int ptid = tid - 5 * 32;
    const int c = ptid % CPR, r0 = ptid / CPR;
    const uint32_t dst_c = static_cast<uint32_t>(c >> 3) * Cfg::SLAB_BYTES;
    int t = 0;
    bool ok = true;
    auto emit = [&](bool is_v, int j) -> bool {
      const int slot = t % SLOTS;
      if (t >= SLOTS && !warp_wait(bar_empty(slot), ((t / SLOTS) - 1) & 1, s_abort, tmo, lane)) return false;
      const int pos0 = (blk0 + j) * PT_KEYS;
      const uint32_t base = ring + slot * Cfg::TILE_BYTES + dst_c;
#pragma unroll
      for (int pass = 0; pass < PT_KEYS / RSTEP; ++pass) {
        const int r = r0 + pass * RSTEP, pos = pos0 + r;
        const __nv_bfloat16 *src = P.q;
        bool have = false;
#pragma unroll
        for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
          const int rr = pos - P.first[sg];
          if (rr >= 0 && rr < P.len[sg]) {
            src = (is_v ? P.v[sg] : P.k[sg]) + static_cast<size_t>(rr) * P.stride[sg] + static_cast<size_t>(kvh) * D_HEAD + c * 8;
            have = true;
          }
        }
        cp_async16(base + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, have);
      }
      cp_async_commit();
      if (t >= PT_LAG) {
        // the block issued PT_LAG blocks ago has landed: publish it to the tensor cores' view of shared memory
        cp_async_wait_group<PT_LAG>();
        fence_proxy_async_smem();
        mbar_arrive(bar_full((t - PT_LAG) % SLOTS));
      }
      ++t;
      return true;
    };
    if (n_blk > 0) {
      ok = emit(false, 0);
      for (int j = 0; ok && j < n_blk; ++j) {
        if (j + 1 < n_blk) ok = emit(false, j + 1);
        if (ok) ok = emit(true, j);
      }
      cp_async_wait_all();
      if (ok) {
        fence_proxy_async_smem();
        for (int u = t > PT_LAG ? t - PT_LAG : 0; u < t; ++u) mbar_arrive(bar_full(u % SLOTS));
      } else {
        raise(P.status, STATUS_TIMEOUT, s_abort);
      }
    }
  }

  // ---- teardown: every role is done with tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::COLS);
  }
}

template <int D_HEAD, int G>
static kvd_status prefill_tc_launch(kvd_ctx *ctx, const PrefillParams &P, cudaStream_t stream) {
  using Cfg = PtCfg<D_HEAD>;
  constexpr int GP = G == 3 ? 4 : G;
  auto k0 = kvd_prefill_attn_tc_kernel<D_HEAD, G, 0>;
  auto k1 = kvd_prefill_attn_tc_kernel<D_HEAD, G, 1>;
  static bool configured[64] = {};
  if (!configured[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(k0, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(prefill attention)");
    configured[ctx->device & 63] = true;
  }
  const int tok = PT_ROWS / GP;
  dim3 grid((P.n_rows + tok - 1) / tok, P.n_kv, 1);
  if (ctx->dtype == 1) k1<<<grid, PT_THREADS, Cfg::SMEM_BYTES, stream>>>(P);
  else k0<<<grid, PT_THREADS, Cfg::SMEM_BYTES, stream>>>(P);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prefill attention");
  ctx->launches += 1;
  return KVD_OK;
}

template <int D_HEAD>
static kvd_status prefill_tc_group(kvd_ctx *ctx, const PrefillParams &P, int group, cudaStream_t stream) {
  switch (group) {
    case 1: return prefill_tc_launch<D_HEAD, 1>(ctx, P, stream);
    case 2: return prefill_tc_launch<D_HEAD, 2>(ctx, P, stream);
    case 3: return prefill_tc_launch<D_HEAD, 3>(ctx, P, stream);
    case 4: return prefill_tc_launch<D_HEAD, 4>(ctx, P, stream);
    case 8: return prefill_tc_launch<D_HEAD, 8>(ctx, P, stream);
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
