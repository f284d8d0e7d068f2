// Fused K/V recomputation kernel (paper Eq. 13-14 with Eq. 1-2 and Eq. 11-12 folded in).
//
//   Y[M, 2*n_kv*d_head] = X[M, d_hidden] * W'          W' = diag(gamma) W_kv, bf16, K-major
//   y <- y / sqrt(mean_i x_i^2 + eps)                   RMSNorm applied after the contraction
//   K heads: optional RMS norm over d_head, scale gamma_k, rotation by the row's position
//   K, V stored as bf16
//
// One persistent CTA per SM walks over 128 x BLOCK_N output tiles.  Warp roles:
//   warp 0      TMA producer: 128x64 tile of X and BLOCK_Nx64 tile of W' per pipeline stage
//   warp 1      owns TMEM; one lane issues tcgen05.mma (128 x BLOCK_N x 16 per instruction)
//   warps 2-5   row statistics: each thread sums x^2 of one row from the X tiles as they land
//   warps 6-9   epilogue: tcgen05.ld the fp32 accumulator, normalise, rotate, convert, store
// The accumulator is double-buffered in TMEM (2 x BLOCK_N columns) so the epilogue of tile i
// overlaps the main loop of tile i+1.
//
// Bit-reproducibility: the k loop always runs over all of d_hidden in ascending order with one MMA
// shape, row sums are taken thread-locally in ascending channel order, the key norm is reduced by
// the single thread that owns the row, and cos/sin depend on (position, channel) only.  A row's
// output bits are therefore independent of M and of the row's index.
#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

template <int BLOCK_N, int D_HEAD>
struct RcCfg {
  static constexpr int STAGES = BLOCK_N == 256 ? 4 : 6;
  static constexpr int A_BYTES = RC_BLOCK_M * RC_BLOCK_K * 2;
  static constexpr int B_BYTES = BLOCK_N * RC_BLOCK_K * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BLOCK_N;
  // barriers: full[S], empty[S], tmem_full[2], tmem_empty[2], stats_full[2]
  static constexpr int NUM_BARS = 2 * STAGES + 6;
  static constexpr int ROPE_LO_BYTES = (D_HEAD / 2) * ROPE_LO_SIZE * 8;  // [pair][position low bits] (cos, sin)
  static constexpr int TAIL_BYTES =
      NUM_BARS * 8 + 16 /*tmem ptr, abort*/ + 2 * RC_BLOCK_M * 4 /*rstd*/ + 256 * 4 /*gamma_k*/ + ROPE_LO_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + TAIL_BYTES + 1024 /*alignment slack*/;
};

// Optional per-tile timeline (SM clock cycles) for performance analysis; see kvd_set_trace.
__device__ __forceinline__ void trace_put(long long *trace, int tile_iter, int field, long long v) {
  if (trace != nullptr && tile_iter < RC_TRACE_TILES)
    trace[(static_cast<size_t>(blockIdx.x) * RC_TRACE_TILES + tile_iter) * RC_TRACE_FIELDS + field] = v;
}

__device__ __forceinline__ void raise(int *status, int bit, volatile int *abort_flag) {
  atomicOr(status, bit);
  *abort_flag = 1;
}

template <int BLOCK_N, int D_HEAD>
__global__ void __launch_bounds__(RC_THREADS, 1)
kvd_recompute_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const RecomputeParams p) {
  using Cfg = RcCfg<BLOCK_N, D_HEAD>;
  constexpr int STAGES = Cfg::STAGES;
  static_assert(BLOCK_N % D_HEAD == 0, "a tile must hold whole heads");

  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *tail = smem + STAGES * Cfg::STAGE_BYTES;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tail);
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(tail + Cfg::NUM_BARS * 8);
  volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);
  float *s_rstd = reinterpret_cast<float *>(tail + Cfg::NUM_BARS * 8 + 16);
  float *s_gamma_k = s_rstd + 2 * RC_BLOCK_M;
  float2 *s_rope_lo = reinterpret_cast<float2 *>(s_gamma_k + 256);

  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(bars);
  auto bar_full = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto bar_tmem_full = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto bar_tmem_empty = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  auto bar_stats_full = [&](int a) { return bar_base + 8u * (2 * STAGES + 4 + a); };

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_tiles = p.num_m_blocks * p.num_n_blocks;
  // Tile order: all key tiles first, then all value tiles, so that the last tile of a CTA (whose
  // epilogue nothing overlaps) is a cheap value tile.  Falls back to row-major order when a tile
  // mixes key and value heads.
  const int nk_tiles = (p.k_cols % BLOCK_N == 0) ? p.k_cols / BLOCK_N : 0;
  auto tile_coords = [&](int t, int &m0, int &n0) {
    if (nk_tiles == 0) {
      m0 = (t / p.num_n_blocks) * RC_BLOCK_M;
      n0 = (t % p.num_n_blocks) * BLOCK_N;
    } else if (t < p.num_m_blocks * nk_tiles) {
      m0 = (t / nk_tiles) * RC_BLOCK_M;
      n0 = (t % nk_tiles) * BLOCK_N;
    } else {
      const int u = t - p.num_m_blocks * nk_tiles, nv = p.num_n_blocks - nk_tiles;
      m0 = (u / nv) * RC_BLOCK_M;
      n0 = (nk_tiles + u % nv) * BLOCK_N;
    }
  };
  const unsigned long long tmo = p.timeout_ns;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1 + 4);  // MMA commit + one arrival per statistics warp
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tmem_full(a), 1);
      mbar_init(bar_tmem_empty(a), 4);          // one arrival per epilogue warp
      mbar_init(bar_stats_full(a), RC_BLOCK_M);  // one arrival per statistics thread
    }
    *s_abort = 0;
    fence_mbar_init();
    prefetch_tensormap(&tmap_a);
    prefetch_tensormap(&tmap_b);
  }
  if (threadIdx.x < D_HEAD) s_gamma_k[threadIdx.x] = p.gamma_k ? p.gamma_k[threadIdx.x] : 1.0f;
  for (int i = threadIdx.x; i < Cfg::ROPE_LO_BYTES / 16; i += RC_THREADS)
    reinterpret_cast<float4 *>(s_rope_lo)[i] = reinterpret_cast<const float4 *>(p.rope_lo)[i];
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  if (threadIdx.x == 0) trace_put(p.trace, 0, 11, clock64());

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      uint32_t issued = 0, issued_parity = 0;  // per-stage: a load is in flight with this parity
      bool ok = true;
      int ti = 0;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++ti) {
        int m0, n0;
        tile_coords(t, m0, n0);
        long long waited = 0;
        trace_put(p.trace, ti, 1, clock64());
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          const long long w0 = p.trace ? clock64() : 0;
          if (!mbar_wait(bar_empty(s), ph ^ 1u, s_abort, tmo)) {
            raise(p.status, STATUS_TIMEOUT, s_abort);
            ok = false;
            break;
          }
          if (p.trace) waited += clock64() - w0;
          mbar_arrive_expect_tx(bar_full(s), Cfg::STAGE_BYTES);
          const uint32_t a_dst = smem_base + s * Cfg::STAGE_BYTES;
          tma_load_2d(a_dst, &tmap_a, bar_full(s), kb * RC_BLOCK_K, m0);
          tma_load_2d(a_dst + Cfg::A_BYTES, &tmap_b, bar_full(s), kb * RC_BLOCK_K, n0);
          issued |= 1u << s;
          issued_parity = (issued_parity & ~(1u << s)) | (ph << s);
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        trace_put(p.trace, ti, 0, waited);
        trace_put(p.trace, ti, 2, clock64());
      }
      if (!ok) {
        // leave no bulk copy in flight behind us: wait (bounded) for every load already issued
        for (int i = 0; i < STAGES; ++i) {
          if (issued & (1u << i)) {
            const unsigned long long t0 = globaltimer_ns();
            while (!mbar_try_wait(bar_full(i), (issued_parity >> i) & 1u)) {
              if (globaltimer_ns() - t0 > 100000000ull) break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(RC_BLOCK_M, BLOCK_N);
      int s = 0, a = 0;
      uint32_t ph = 0, aph = 0;
      bool ok = true;
      int ti = 0;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++ti) {
        if (!mbar_wait(bar_tmem_empty(a), aph ^ 1u, s_abort, tmo)) {
          raise(p.status, STATUS_TIMEOUT, s_abort);
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BLOCK_N;
        long long waited = 0;
        trace_put(p.trace, ti, 4, clock64());
        trace_put(p.trace, ti, 10, t);
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          const long long w0 = p.trace ? clock64() : 0;
          if (!mbar_wait(bar_full(s), ph, s_abort, tmo)) {
            raise(p.status, STATUS_TIMEOUT, s_abort);
            ok = false;
            break;
          }
          if (p.trace) waited += clock64() - w0;
          tc_fence_after();
          const uint32_t a_addr = smem_base + s * Cfg::STAGE_BYTES;
          const uint64_t a_desc = umma_smem_desc_sw128(a_addr);
          const uint64_t b_desc = umma_smem_desc_sw128(a_addr + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < RC_BLOCK_K / 16; ++k) {
            // 16 bf16 = 32 bytes along K inside the 128-byte swizzle row: +2 in the address field
            umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(bar_empty(s));
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (!ok) break;
        umma_commit(bar_tmem_full(a));
        trace_put(p.trace, ti, 3, waited);
        trace_put(p.trace, ti, 5, clock64());
        if (++a == 2) {
          a = 0;
          aph ^= 1u;
        }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ row statistics (Eq. 2)
    const int row = (warp - 2) * 32 + lane;
    const uint32_t row_off = row * 128u;
    const uint32_t sw = (row & 7u) << 4;
    int s = 0, a = 0;
    uint32_t ph = 0, aph = 0;
    bool ok = true;
    int ti = 0;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++ti) {
      long long waited = 0;
      const long long st0 = p.trace ? clock64() : 0;
      // s_rstd[a] is free once the epilogue that read it released accumulator a
      // the whole warp takes the same branch: aligned instructions follow
      if (!__all_sync(0xffffffffu, mbar_wait(bar_tmem_empty(a), aph ^ 1u, s_abort, tmo))) {
        raise(p.status, STATUS_TIMEOUT, s_abort);
        break;
      }
      // eight partial sums (one per element slot of a 16-byte chunk) keep the FMA chains short; they
      // are combined in a fixed order below, the same for every row
      float ps[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int kb = 0; kb < p.num_k_blocks; ++kb) {
        const long long w0 = p.trace ? clock64() : 0;
        if (!__all_sync(0xffffffffu, mbar_wait(bar_full(s), ph, s_abort, tmo))) {
          raise(p.status, STATUS_TIMEOUT, s_abort);
          ok = false;
          break;
        }
        if (p.trace) waited += clock64() - w0;
        const uint32_t a_addr = smem_base + s * Cfg::STAGE_BYTES + row_off;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          // logical 16-byte chunk c of this row sits at chunk (c ^ (row % 8)) under the 128-byte swizzle
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                       : "r"(a_addr + ((static_cast<uint32_t>(c) << 4) ^ sw)));
          float x;
          x = bf16_lo(w0); ps[0] = fmaf(x, x, ps[0]);
          x = bf16_hi(w0); ps[1] = fmaf(x, x, ps[1]);
          x = bf16_lo(w1); ps[2] = fmaf(x, x, ps[2]);
          x = bf16_hi(w1); ps[3] = fmaf(x, x, ps[3]);
          x = bf16_lo(w2); ps[4] = fmaf(x, x, ps[4]);
          x = bf16_hi(w2); ps[5] = fmaf(x, x, ps[5]);
          x = bf16_lo(w3); ps[6] = fmaf(x, x, ps[6]);
          x = bf16_hi(w3); ps[7] = fmaf(x, x, ps[7]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty(s));
        if (++s == STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (!ok) break;
      const float sum = ((ps[0] + ps[1]) + (ps[2] + ps[3])) + ((ps[4] + ps[5]) + (ps[6] + ps[7]));
      s_rstd[a * RC_BLOCK_M + row] = 1.0f / sqrtf(sum * p.inv_d_hidden + p.rms_eps);
      mbar_arrive(bar_stats_full(a));
      if (threadIdx.x == 64) {
        trace_put(p.trace, ti, 8, waited);
        trace_put(p.trace, ti, 9, clock64() - st0);
      }
      if (++a == 2) {
        a = 0;
        aph ^= 1u;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32) belong to this warp
    const int row = quarter * 32 + lane;
    const uint32_t lane_field = static_cast<uint32_t>(quarter * 32) << 16;
    constexpr int HALF = D_HEAD / 2;
    int a = 0;
    uint32_t aph = 0;
    int ti = 0;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++ti) {
      int m0, n0;
      tile_coords(t, m0, n0);
      const bool ready = mbar_wait(bar_tmem_full(a), aph, s_abort, tmo) && mbar_wait(bar_stats_full(a), aph, s_abort, tmo);
      if (!__all_sync(0xffffffffu, ready)) {  // warp-uniform: tcgen05.ld below is an aligned instruction
        raise(p.status, STATUS_TIMEOUT, s_abort);
        break;
      }
      tc_fence_after();
      if (threadIdx.x == 6 * 32) trace_put(p.trace, ti, 6, clock64());
      const int m = m0 + row;
      const bool valid = m < p.M;
      const float rstd = s_rstd[a * RC_BLOCK_M + row];
      int pos = valid ? p.positions[m] : 0;
      if (pos < 0 || pos >= p.max_pos) {
        atomicOr(p.status, STATUS_POSITION);
        pos = pos < 0 ? 0 : p.max_pos - 1;
      }
      // (cos, sin) of pos * f_i = angle sum of the entries for (pos & ~15) [global, shared by 16
      // neighbouring positions] and (pos & 15) [shared memory, laid out [pair][low bits]]
      const float4 *t_hi = reinterpret_cast<const float4 *>(p.rope_hi + static_cast<size_t>(pos >> ROPE_LO_BITS) * HALF);
      const float2 *t_lo = s_rope_lo + (pos & (ROPE_LO_SIZE - 1));
      const uint32_t acc = tmem_base + lane_field + a * BLOCK_N;

#pragma unroll 1
      for (int hh = 0; hh < BLOCK_N / D_HEAD; ++hh) {
        const int col0 = n0 + hh * D_HEAD;  // first fused column of this head
        const uint32_t tcol = acc + hh * D_HEAD;
        if (col0 >= p.k_cols) {
          // ---- value head (Eq. 14): scale by 1/rms and store
          __nv_bfloat16 *dst = p.v_out + static_cast<size_t>(m) * p.out_row_stride + (col0 - p.k_cols);
#pragma unroll 1
          for (int c = 0; c < D_HEAD / 32; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tcol + c * 32, r);
            tmem_wait_ld();
            uint32_t o[16];
#pragma unroll
            for (int j = 0; j < 16; ++j)
              o[j] = pack_bf16(__uint_as_float(r[2 * j]) * rstd, __uint_as_float(r[2 * j + 1]) * rstd);
            if (valid) {
              uint4 *d4 = reinterpret_cast<uint4 *>(dst + c * 32);
#pragma unroll
              for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
            }
          }
        } else {
          // ---- key head (Eq. 13): 1/rms, optional key norm, rotation R_pos
          __nv_bfloat16 *dst = p.k_out + static_cast<size_t>(m) * p.out_row_stride + col0;
          float kscale = rstd;
          if (p.qk_norm) {
            float ss = 0.f;
#pragma unroll 1
            for (int c = 0; c < D_HEAD / 32; ++c) {
              uint32_t r[32];
              tmem_ld_x32(tcol + c * 32, r);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float v = __uint_as_float(r[j]) * rstd;
                ss = fmaf(v, v, ss);
              }
            }
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
              uint32_t o[8];
#pragma unroll
              for (int j = 0; j < 8; j += 2) {
                const int i = c * 8 + j;  // pairs i and i + 1
                const float2 l0 = t_lo[i * ROPE_LO_SIZE], l1 = t_lo[(i + 1) * ROPE_LO_SIZE];
                const float4 hh4 = h[j >> 1];
                const float c0 = fmaf(hh4.x, l0.x, -hh4.y * l0.y), s0 = fmaf(hh4.y, l0.x, hh4.x * l0.y);
                const float c1 = fmaf(hh4.z, l1.x, -hh4.w * l1.y), s1 = fmaf(hh4.w, l1.x, hh4.z * l1.y);
                const float a0 = __uint_as_float(r[2 * j]) * kscale * s_gamma_k[c * 16 + 2 * j];
                const float b0 = __uint_as_float(r[2 * j + 1]) * kscale * s_gamma_k[c * 16 + 2 * j + 1];
                const float a1 = __uint_as_float(r[2 * j + 2]) * kscale * s_gamma_k[c * 16 + 2 * j + 2];
                const float b1 = __uint_as_float(r[2 * j + 3]) * kscale * s_gamma_k[c * 16 + 2 * j + 3];
                o[j] = pack_bf16(fmaf(a0, c0, -b0 * s0), fmaf(a0, s0, b0 * c0));
                o[j + 1] = pack_bf16(fmaf(a1, c1, -b1 * s1), fmaf(a1, s1, b1 * c1));
              }
              if (valid) {
                uint4 *d4 = reinterpret_cast<uint4 *>(dst + c * 16);
                d4[0] = make_uint4(o[0], o[1], o[2], o[3]);
                d4[1] = make_uint4(o[4], o[5], o[6], o[7]);
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
              uint32_t oa[8], ob[8];
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                const int i = c * 16 + j;  // pairs (i, i + HALF) and (i + 1, i + 1 + HALF)
                const float2 l0 = t_lo[i * ROPE_LO_SIZE], l1 = t_lo[(i + 1) * ROPE_LO_SIZE];
                const float4 hh4 = h[j >> 1];
                const float c0 = fmaf(hh4.x, l0.x, -hh4.y * l0.y), s0 = fmaf(hh4.y, l0.x, hh4.x * l0.y);
                const float c1 = fmaf(hh4.z, l1.x, -hh4.w * l1.y), s1 = fmaf(hh4.w, l1.x, hh4.z * l1.y);
                const float a0 = __uint_as_float(ra[j]) * kscale * s_gamma_k[i];
                const float b0 = __uint_as_float(rb[j]) * kscale * s_gamma_k[i + HALF];
                const float a1 = __uint_as_float(ra[j + 1]) * kscale * s_gamma_k[i + 1];
                const float b1 = __uint_as_float(rb[j + 1]) * kscale * s_gamma_k[i + 1 + HALF];
                oa[j >> 1] = pack_bf16(fmaf(a0, c0, -b0 * s0), fmaf(a1, c1, -b1 * s1));
                ob[j >> 1] = pack_bf16(fmaf(a0, s0, b0 * c0), fmaf(a1, s1, b1 * c1));
              }
              if (valid) {
                uint4 *da = reinterpret_cast<uint4 *>(dst + c * 16);
                uint4 *db = reinterpret_cast<uint4 *>(dst + HALF + c * 16);
                da[0] = make_uint4(oa[0], oa[1], oa[2], oa[3]);
                da[1] = make_uint4(oa[4], oa[5], oa[6], oa[7]);
                db[0] = make_uint4(ob[0], ob[1], ob[2], ob[3]);
                db[1] = make_uint4(ob[4], ob[5], ob[6], ob[7]);
              }
            }
          }
        }
      }
      // accumulator a (and s_rstd[a]) may be overwritten now
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tmem_empty(a));
      if (threadIdx.x == 6 * 32) trace_put(p.trace, ti, 7, clock64());
      if (++a == 2) {
        a = 0;
        aph ^= 1u;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------ host launcher
template <int BLOCK_N, int D_HEAD>
static kvd_status launch_impl(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_a, const RecomputeParams &p,
                              cudaStream_t stream) {
  using Cfg = RcCfg<BLOCK_N, D_HEAD>;
  auto kern = kvd_recompute_kernel<BLOCK_N, D_HEAD>;
  static bool configured[64] = {};
  if (!configured[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(recompute)");
    configured[ctx->device & 63] = true;
  }
  const int tiles = p.num_m_blocks * p.num_n_blocks;
  const int grid = tiles < ctx->num_sms ? tiles : ctx->num_sms;
  kern<<<grid, RC_THREADS, Cfg::SMEM_BYTES, stream>>>(tmap_a, ls.tmap_b, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch recompute");
  ctx->launches += 1;
  return KVD_OK;
}

kvd_status launch_recompute(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_a, const RecomputeParams &p,
                            cudaStream_t stream) {
  const int dh = ctx->desc.d_head;
  if (ctx->block_n == 256) {
    if (dh == 256) return launch_impl<256, 256>(ctx, ls, tmap_a, p, stream);
    if (dh == 128) return launch_impl<256, 128>(ctx, ls, tmap_a, p, stream);
    if (dh == 64) return launch_impl<256, 64>(ctx, ls, tmap_a, p, stream);
  } else if (ctx->block_n == 128) {
    if (dh == 128) return launch_impl<128, 128>(ctx, ls, tmap_a, p, stream);
    if (dh == 64) return launch_impl<128, 64>(ctx, ls, tmap_a, p, stream);
  }
  return KVD_ERR_SHAPE;
}

}  // namespace kvd
