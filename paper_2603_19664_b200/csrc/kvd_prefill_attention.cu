// ATTENTION of Algorithm 1 (Eq. 6-7) for MANY query tokens of one sequence, each with its own causal limit: the
// prefill-shaped call (a user segment processed at once; the replay of an evicted prefix when only one residual row
// per token is kept).  Tiled over query rows on the tensor cores (mma.sync m16n8k16, fp32 accumulation):
//
//   CTA = (tile of query tokens, KV head), four warps, 64 MMA rows = 64 / Gp tokens x Gp query heads of the group
//         (Gp = group size rounded up to a power of two; padding heads are zero rows that are never stored);
//   keys are taken in blocks of 64 aligned to ABSOLUTE position, gathered from the segments into shared memory
//         (cp.async, 16-byte chunks, xor-swizzled for ldmatrix), S = Q K^T, mask (position <= the row's own, inside the
//         window, key present), online softmax in base 2, P rounded to the element type, O += P V.
//
// A row's result depends on that row alone: every row walks the key blocks of its tile in ascending order, a block
// without a visible key for the row changes nothing for it (weights 0, rescale by exactly 1), the block boundaries
// are absolute, and mma.sync computes output rows independently.  So a token attended alone and the same token
// inside any tile give the same bits -- which is what a replay in other batch sizes needs.  The bits are NOT those
// of kvd_decode_attention (another split, P rounded before the second product): same tolerance against the
// definition, and callers that need bit-identical outputs across cache policies use one of the two calls throughout.
#include <math_constants.h>
#include <stdlib.h>
#include <string.h>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

constexpr int PF_BLOCK_KEYS = 64;
constexpr int PF_ROWS = 64;  // MMA rows per CTA


__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
template <int DT>
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  if constexpr (DT == 0)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  else
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// byte offset of 16-byte chunk `c` of row `r` in a tile whose rows hold D_HEAD 16-bit elements, the low three bits
// of the chunk index xor-ed with the row so that the eight rows of an ldmatrix read hit eight different banks groups
template <int D_HEAD>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return static_cast<uint32_t>(r) * (D_HEAD * 2) + static_cast<uint32_t>(((c & ~7) | ((c ^ r) & 7)) * 16);
}

template <int D_HEAD, int G, int DT>
__global__ void __launch_bounds__(128) kvd_prefill_attn_kernel(const __grid_constant__ PrefillParams P) {
  constexpr int GP = G == 3 ? 4 : G;       // heads of the group, padded to a power of two
  constexpr int TOK = PF_ROWS / GP;        // query tokens per CTA
  constexpr int CH = D_HEAD / 8;           // 16-byte chunks per row
  constexpr int KT = D_HEAD / 16;          // k steps of the first product, channel-tile pairs of the second
  constexpr int TILE = PF_ROWS * D_HEAD * 2;
  extern __shared__ __align__(128) uint8_t pf_smem[];
  __shared__ int s_lo, s_hi;
  const uint32_t q_s = smem_u32(pf_smem), k_s = q_s + TILE, v_s = k_s + TILE;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * TOK, kvh = blockIdx.y;
  grid_launch_dependents();
  if (tid == 0) {
    s_lo = INT_MAX;
    s_hi = -1;
  }
  grid_dependency_wait();
  __syncthreads();

  // ---- the tile's queries into shared memory (MMA row m = token m / GP, head m % GP of the group)
  for (int idx = tid; idx < PF_ROWS * CH; idx += 128) {
    const int m = idx / CH, c = idx % CH;
    const int tok = tok0 + m / GP, g = m % GP;
    const bool ok = tok < P.n_rows && g < G;
    const __nv_bfloat16 *src = ok ? P.q + (static_cast<size_t>(tok) * P.n_q + kvh * G + g) * D_HEAD + c * 8 : P.q;
    cp_async16(q_s + tile_off<D_HEAD>(m, c), src, ok);
  }
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
  // this thread's two accumulator rows
  const int r0 = warp * 16 + (lane >> 2), r1 = r0 + 8;
  const int t0 = tok0 + r0 / GP, t1 = tok0 + r1 / GP;
  const int qp0 = t0 < P.n_rows ? P.q_pos[t0] : -1, qp1 = t1 < P.n_rows ? P.q_pos[t1] : -1;
  const int lo0 = P.window > 0 ? qp0 - P.window + 1 : 0, lo1 = P.window > 0 ? qp1 - P.window + 1 : 0;
  __syncthreads();
  const int blk0 = s_hi >= 0 ? s_lo / PF_BLOCK_KEYS : 0, blk1 = s_hi >= 0 ? s_hi / PF_BLOCK_KEYS : -1;

  float o[CH][4];
#pragma unroll
  for (int i = 0; i < CH; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
  float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};

  for (int blk = blk0; blk <= blk1; ++blk) {
    const int pos0 = blk * PF_BLOCK_KEYS;
    __syncthreads();  // the previous block's fragments have been read
    // ---- gather the block's keys and values (a position no segment holds reads as zeros and is masked below)
    for (int idx = tid; idx < PF_BLOCK_KEYS * CH; idx += 128) {
      const int j = idx / CH, c = idx % CH;
      const int pos = pos0 + j;
      const __nv_bfloat16 *kp = P.q, *vp = P.q;
      bool ok = false;
#pragma unroll
      for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
        const int r = pos - P.first[sg];
        if (r >= 0 && r < P.len[sg]) {
          const size_t off = static_cast<size_t>(r) * P.stride[sg] + static_cast<size_t>(kvh) * D_HEAD + c * 8;
          kp = P.k[sg] + off;
          vp = P.v[sg] + off;
          ok = true;
        }
      }
      cp_async16(k_s + tile_off<D_HEAD>(j, c), kp, ok);
      cp_async16(v_s + tile_off<D_HEAD>(j, c), vp, ok);
    }
    cp_async_wait_all();
    __syncthreads();

    // ---- S = Q K^T for this warp's 16 rows and the block's 64 keys
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[nt][j] = 0.f;
#pragma unroll 4
    for (int kk = 0; kk < KT; ++kk) {
      uint32_t a[4];
      {
        const int mat = lane >> 3, rr = lane & 7;
        ldsm_x4(q_s + tile_off<D_HEAD>(warp * 16 + rr + (mat & 1) * 8, 2 * kk + (mat >> 1)), a);
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {  // pairs of key tiles
        uint32_t b[4];
        const int mat = lane >> 3, rr = lane & 7;
        ldsm_x4(k_s + tile_off<D_HEAD>(np * 16 + rr + (mat >> 1) * 8, 2 * kk + (mat & 1)), b);
        mma_16816<DT>(s[2 * np], a, b[0], b[1]);
        mma_16816<DT>(s[2 * np + 1], a, b[2], b[3]);
      }
    }
    // ---- mask, online softmax (log2 units)
    float bm[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pos = pos0 + nt * 8 + (lane & 3) * 2 + (j & 1);
        const int qp = (j & 2) ? qp1 : qp0, lo = (j & 2) ? lo1 : lo0;
        bool present = false;
#pragma unroll
        for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) present |= (pos - P.first[sg] >= 0 && pos - P.first[sg] < P.len[sg]);
        const bool vis = present && pos <= qp && pos >= lo;
        s[nt][j] = vis ? s[nt][j] * P.scale_log2e : -CUDART_INF_F;
        bm[j >> 1] = fmaxf(bm[j >> 1], s[nt][j]);
      }
    }
    float corr[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      bm[h] = fmaxf(bm[h], __shfl_xor_sync(0xffffffffu, bm[h], 1));
      bm[h] = fmaxf(bm[h], __shfl_xor_sync(0xffffffffu, bm[h], 2));
      const float m_new = fmaxf(m_run[h], bm[h]);
      const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
      corr[h] = exp2f(m_run[h] - m_use);  // 0 while nothing has been seen, exactly 1 when the maximum stays
      m_run[h] = m_new;
      l_run[h] *= corr[h];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        s[nt][2 * h] = exp2f(s[nt][2 * h] - m_use);
        s[nt][2 * h + 1] = exp2f(s[nt][2 * h + 1] - m_use);
      }
    }
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      o[i][0] *= corr[0];
      o[i][1] *= corr[0];
      o[i][2] *= corr[1];
      o[i][3] *= corr[1];
    }
    // ---- O += P V, P rounded to the element type (the rounded weights are also what the row sum adds up)
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      uint32_t a[4];
      a[0] = pack_out<DT>(s[2 * ks][0], s[2 * ks][1]);
      a[1] = pack_out<DT>(s[2 * ks][2], s[2 * ks][3]);
      a[2] = pack_out<DT>(s[2 * ks + 1][0], s[2 * ks + 1][1]);
      a[3] = pack_out<DT>(s[2 * ks + 1][2], s[2 * ks + 1][3]);
      {
        float p0, p1;
        unpack2(x2_to_f32x2<DT>(a[0]), p0, p1);
        l_run[0] += p0 + p1;
        unpack2(x2_to_f32x2<DT>(a[2]), p0, p1);
        l_run[0] += p0 + p1;
        unpack2(x2_to_f32x2<DT>(a[1]), p0, p1);
        l_run[1] += p0 + p1;
        unpack2(x2_to_f32x2<DT>(a[3]), p0, p1);
        l_run[1] += p0 + p1;
      }
#pragma unroll
      for (int ct = 0; ct < KT; ++ct) {  // pairs of channel tiles
        uint32_t b[4];
        const int mat = lane >> 3, rr = lane & 7;
        ldsm_x4_trans(v_s + tile_off<D_HEAD>(ks * 16 + rr + (mat & 1) * 8, 2 * ct + (mat >> 1)), b);
        mma_16816<DT>(o[2 * ct], a, b[0], b[1]);
        mma_16816<DT>(o[2 * ct + 1], a, b[2], b[3]);
      }
    }
  }

  // ---- normalise and store (a token without a visible key yields zeros)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = h == 0 ? r0 : r1, tok = h == 0 ? t0 : t1, g = r % GP;
    if (tok >= P.n_rows || g >= G) continue;
    const float inv = l_run[h] > 0.f ? 1.0f / l_run[h] : 0.f;
    uint32_t *dst = reinterpret_cast<uint32_t *>(P.out + (static_cast<size_t>(tok) * P.n_q + kvh * G + g) * D_HEAD) + (lane & 3);
#pragma unroll
    for (int i = 0; i < CH; ++i) dst[i * 4] = pack_out<DT>(o[i][2 * h] * inv, o[i][2 * h + 1] * inv);
  }
}

template <int D_HEAD, int G>
static kvd_status prefill_launch(kvd_ctx *ctx, const PrefillParams &P, cudaStream_t stream) {
  constexpr int GP = G == 3 ? 4 : G;
  constexpr int SMEM = 3 * PF_ROWS * D_HEAD * 2;
  auto k0 = kvd_prefill_attn_kernel<D_HEAD, G, 0>;
  auto k1 = kvd_prefill_attn_kernel<D_HEAD, G, 1>;
  static bool configured[64] = {};
  if (!configured[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(k0, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(prefill attention)");
    configured[ctx->device & 63] = true;
  }
  const int tok = PF_ROWS / GP;
  dim3 grid((P.n_rows + tok - 1) / tok, P.n_kv, 1);
  if (ctx->dtype == 1) k1<<<grid, 128, SMEM, stream>>>(P);
  else k0<<<grid, 128, SMEM, stream>>>(P);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch prefill attention");
  ctx->launches += 1;
  return KVD_OK;
}

template <int D_HEAD>
static kvd_status prefill_group(kvd_ctx *ctx, const PrefillParams &P, int group, cudaStream_t stream) {
  switch (group) {
    case 1: return prefill_launch<D_HEAD, 1>(ctx, P, stream);
    case 2: return prefill_launch<D_HEAD, 2>(ctx, P, stream);
    case 3: return prefill_launch<D_HEAD, 3>(ctx, P, stream);
    case 4: return prefill_launch<D_HEAD, 4>(ctx, P, stream);
    case 8: return prefill_launch<D_HEAD, 8>(ctx, P, stream);
    default: return KVD_ERR_SHAPE;
  }
}

}  // namespace kvd

using namespace kvd;

extern "C" kvd_status kvd_prefill_attention(kvd_ctx *ctx, int layer, int n_rows, const void *q, const int32_t *q_pos,
                                            const kvd_kv_segment *segs, int n_segs, float scale, void *out, void *stream_) {
  if (!ctx || n_rows < 0 || n_segs < 0 || n_segs > KVD_MAX_SEGMENTS) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (ctx->dtype == KVD_DTYPE_F32) return KVD_ERR_UNSUPPORTED;
  if (n_rows == 0) return KVD_OK;
  if (!q || !q_pos || !out || (n_segs > 0 && !segs)) return KVD_ERR_INVALID_ARG;
  if (((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) & 15u) != 0) return KVD_ERR_ALIGNMENT;
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  static thread_local PrefillParams P;
  P.seg_lo = INT32_MAX;
  P.seg_hi = -1;
  for (int s = 0; s < KVD_MAX_SEGMENTS; ++s) {
    P.k[s] = P.v[s] = nullptr;
    P.stride[s] = 0;
    P.first[s] = 0;
    P.len[s] = 0;
    if (s >= n_segs) continue;
    const kvd_kv_segment &sg = segs[s];
    if (sg.len < 0 || sg.first_pos < 0) return KVD_ERR_INVALID_ARG;
    if (sg.len == 0) continue;
    if (!sg.k || !sg.v || sg.row_stride < kdim) return KVD_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(sg.k) | reinterpret_cast<uintptr_t>(sg.v)) & 15u) != 0 || sg.row_stride % 8 != 0) return KVD_ERR_ALIGNMENT;
    if (static_cast<int64_t>(sg.first_pos) + sg.len > INT32_MAX) return KVD_ERR_INVALID_ARG;
    for (int s2 = 0; s2 < s; ++s2)
      if (segs[s2].len > 0 && sg.first_pos < segs[s2].first_pos + segs[s2].len && segs[s2].first_pos < sg.first_pos + sg.len)
        return KVD_ERR_INVALID_ARG;
    P.k[s] = static_cast<const __nv_bfloat16 *>(sg.k);
    P.v[s] = static_cast<const __nv_bfloat16 *>(sg.v);
    P.stride[s] = sg.row_stride;
    P.first[s] = sg.first_pos;
    P.len[s] = sg.len;
    if (sg.first_pos < P.seg_lo) P.seg_lo = sg.first_pos;
    if (sg.first_pos + sg.len - 1 > P.seg_hi) P.seg_hi = sg.first_pos + sg.len - 1;
  }
  if (P.seg_hi < 0) P.seg_lo = 0;
  P.q = static_cast<const __nv_bfloat16 *>(q);
  P.out = static_cast<__nv_bfloat16 *>(out);
  P.q_pos = q_pos;
  P.n_rows = n_rows;
  P.n_q = d.n_q_heads;
  P.n_kv = d.n_kv_heads;
  P.window = ls.window;
  P.scale_log2e = (scale > 0.f ? scale : 1.0f / sqrtf(static_cast<float>(d.d_head))) * 1.4426950408889634f;
  P.status = ctx->d_status;
  P.timeout_ns = ctx->timeout_ns;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int group = d.n_q_heads / d.n_kv_heads;
  // the tcgen05 form unless the environment asks for the mma.sync one (comparisons)
  static const bool legacy = getenv("KVD_PREFILL_MMA_SYNC") != nullptr;
  if (!legacy) return launch_prefill_tc(ctx, P, d.d_head, group, stream);
  switch (d.d_head) {
    case 64: return prefill_group<64>(ctx, P, group, stream);
    case 128: return prefill_group<128>(ctx, P, group, stream);
    case 256: return prefill_group<256>(ctx, P, group, stream);
    default: return KVD_ERR_SHAPE;
  }
}
