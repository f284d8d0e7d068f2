// Decode attention (paper Eq. 6-7; ATTENTION(Q, K_all, V_all) of Algorithm 1) for one query token
// per sequence, grouped-query heads, keys given as up to four position-contiguous segments.
//
// Split over keys: the visible position range of a sequence is cut into chunks aligned to absolute
// position.  One CTA handles one (chunk, KV head): it streams that head's K and V rows with
// coalesced 16-byte loads, every lane owning 8 channels, and serves all query heads of the group
// from the same loads.  Scores of 8 keys at a time are reduced across the lanes of a key with a
// transposing shuffle butterfly, the softmax runs online in base 2, and each CTA writes one partial
// (max, sum, unnormalised output) per query head.  A second kernel merges the partials in chunk
// order.
//
// Which chunk, warp, lane group and slot a key lands in is a function of its position only, and the
// merge runs in chunk order, so the output bits do not depend on how the keys are spread over
// segments.
#include <math_constants.h>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

namespace kvd {

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Sum each of the 8 values over the LPK lanes of a group; afterwards the lane whose index bits
// (LPK/2, LPK/4, LPK/8) spell slot u holds the total of v[u].
template <int LPK>
__device__ __forceinline__ float reduce8_transposed(const float (&v)[8], int lig) {
  float w4[4], w2[2], w1;
  {
    const bool up = (lig & (LPK / 2)) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = up ? v[i] : v[i + 4];
      const float keep = up ? v[i + 4] : v[i];
      w4[i] = keep + __shfl_xor_sync(0xffffffffu, send, LPK / 2);
    }
  }
  {
    const bool up = (lig & (LPK / 4)) != 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = up ? w4[i] : w4[i + 2];
      const float keep = up ? w4[i + 2] : w4[i];
      w2[i] = keep + __shfl_xor_sync(0xffffffffu, send, LPK / 4);
    }
  }
  {
    const bool up = (lig & (LPK / 8)) != 0;
    const float send = up ? w2[0] : w2[1];
    const float keep = up ? w2[1] : w2[0];
    w1 = keep + __shfl_xor_sync(0xffffffffu, send, LPK / 8);
  }
#pragma unroll
  for (int m = LPK / 16; m >= 1; m >>= 1) w1 += __shfl_xor_sync(0xffffffffu, w1, m);
  return w1;
}

template <int D_HEAD, int G>
__global__ void __launch_bounds__(AT_THREADS) kvd_attn_split_kernel(const __grid_constant__ AttnLaunch P) {
  constexpr int LPK = D_HEAD / 8;         // lanes per key
  constexpr int KPL = 32 / LPK;           // keys per warp-wide load
  constexpr int U = AT_UNROLL;            // keys per lane group per iteration
  constexpr int NPART = AT_WARPS * KPL;   // lane groups per CTA
  __shared__ float s_o[NPART][G][D_HEAD];
  __shared__ float s_m[NPART][G];
  __shared__ float s_l[NPART][G];

  // ---- which (sequence, chunk) is this CTA's?
  int si = 0;
  {
    int lo = 0, hi = P.n_seqs - 1;
    const int b = blockIdx.x;
    while (lo < hi) {  // last sequence whose first partial index is <= b
      const int mid = (lo + hi + 1) >> 1;
      if (P.seq[mid].part_base - P.seq[0].part_base <= b) lo = mid; else hi = mid - 1;
    }
    si = lo;
  }
  const AttnSeq &S = P.seq[si];
  const int chunk = blockIdx.x - (S.part_base - P.seq[0].part_base);
  const int kvh = blockIdx.y;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int grp = lane / LPK;   // lane group inside the warp
  const int lig = lane % LPK;   // lane inside the group: owns channels [8*lig, 8*lig + 8)
  const int my_slot = ((lig & (LPK / 2)) ? 4 : 0) + ((lig & (LPK / 4)) ? 2 : 0) + ((lig & (LPK / 8)) ? 1 : 0);
  const int chunk_keys = KPL * U * AT_WARPS * S.iters;
  const int chunk_pos0 = S.chunk0_pos + chunk * chunk_keys;

  // ---- query of every head of the group, pre-multiplied by scale * log2(e)
  float qf[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const __nv_bfloat16 *qp = P.q + (static_cast<size_t>(si) * P.n_q + kvh * G + g) * D_HEAD + lig * 8;
    const uint4 w = *reinterpret_cast<const uint4 *>(qp);
    qf[g][0] = bf16_lo(w.x) * P.scale_log2e; qf[g][1] = bf16_hi(w.x) * P.scale_log2e;
    qf[g][2] = bf16_lo(w.y) * P.scale_log2e; qf[g][3] = bf16_hi(w.y) * P.scale_log2e;
    qf[g][4] = bf16_lo(w.z) * P.scale_log2e; qf[g][5] = bf16_hi(w.z) * P.scale_log2e;
    qf[g][6] = bf16_lo(w.w) * P.scale_log2e; qf[g][7] = bf16_hi(w.w) * P.scale_log2e;
  }

  float m_run[G], l_run[G], acc[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_run[g] = -CUDART_INF_F;
    l_run[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[g][e] = 0.f;
  }

  const size_t head_off = static_cast<size_t>(kvh) * D_HEAD + lig * 8;

  for (int it = 0; it < S.iters; ++it) {
    const int pos0 = chunk_pos0 + ((it * AT_WARPS + warp) * KPL + grp) * U;  // this group's 8 positions
    // ---- resolve the 8 keys to addresses (masked keys read a valid dummy row and score -inf)
    const __nv_bfloat16 *kp[U];
    const __nv_bfloat16 *vp[U];
    uint32_t vmask = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int pos = pos0 + u;
      kp[u] = P.q;  // any mapped, 16-byte aligned address
      vp[u] = P.q;
      if (pos >= S.lo_pos && pos <= S.hi_pos) {
#pragma unroll
        for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
          const int r = pos - S.first[sg];
          if (r >= 0 && r < S.len[sg]) {
            const size_t off = static_cast<size_t>(r) * S.stride[sg] + head_off;
            kp[u] = S.k[sg] + off;
            vp[u] = S.v[sg] + off;
            vmask |= 1u << u;
          }
        }
      }
    }
    uint4 kr[U], vr[U];
#pragma unroll
    for (int u = 0; u < U; ++u) kr[u] = ldg_stream(kp[u]);
#pragma unroll
    for (int u = 0; u < U; ++u) vr[u] = ldg_stream(vp[u]);

    // ---- scores: per-lane partial dot products, then the transposing reduction
    float kf[U][8];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      kf[u][0] = bf16_lo(kr[u].x); kf[u][1] = bf16_hi(kr[u].x);
      kf[u][2] = bf16_lo(kr[u].y); kf[u][3] = bf16_hi(kr[u].y);
      kf[u][4] = bf16_lo(kr[u].z); kf[u][5] = bf16_hi(kr[u].z);
      kf[u][6] = bf16_lo(kr[u].w); kf[u][7] = bf16_hi(kr[u].w);
    }
    float pb[G][U];  // softmax numerators of the 8 keys, broadcast to every lane of the group
    float corr[G];
    const bool my_valid = (vmask >> my_slot) & 1u;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float part[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) d = fmaf(qf[g][e], kf[u][e], d);
        part[u] = d;
      }
      float sc = reduce8_transposed<LPK>(part, lig);
      sc = my_valid ? sc : -CUDART_INF_F;
      float bmax = sc;
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, LPK / 2));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, LPK / 4));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, LPK / 8));
      const float m_new = fmaxf(m_run[g], bmax);
      const float m_use = (m_new == -CUDART_INF_F) ? 0.f : m_new;
      const float pmine = exp2f(sc - m_use);  // 0 for masked keys
      corr[g] = exp2f(m_run[g] - m_use);      // 0 while nothing has been seen
      m_run[g] = m_new;
      // every lane with the same slot holds the same pmine; count it once per slot (lanes whose
      // low bits are zero), the group-wide sum is taken at the end
      const bool counts = (lig & (LPK / 8 - 1)) == 0;
      l_run[g] = l_run[g] * corr[g] + (counts ? pmine : 0.f);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int src = grp * LPK + ((u & 4) ? LPK / 2 : 0) + ((u & 2) ? LPK / 4 : 0) + ((u & 1) ? LPK / 8 : 0);
        pb[g][u] = __shfl_sync(0xffffffffu, pmine, src);
      }
    }
    // ---- weighted values
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[g][e] *= corr[g];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float vf[8];
      vf[0] = bf16_lo(vr[u].x); vf[1] = bf16_hi(vr[u].x);
      vf[2] = bf16_lo(vr[u].y); vf[3] = bf16_hi(vr[u].y);
      vf[4] = bf16_lo(vr[u].z); vf[5] = bf16_hi(vr[u].z);
      vf[6] = bf16_lo(vr[u].w); vf[7] = bf16_hi(vr[u].w);
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[g][e] = fmaf(pb[g][u], vf[e], acc[g][e]);
    }
  }

  // ---- combine the lane groups of the CTA in a fixed order
  const int part = warp * KPL + grp;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float l = l_run[g];
    // sum over the lanes of the group (each slot was counted once)
#pragma unroll
    for (int msk = LPK / 2; msk >= 1; msk >>= 1) l += __shfl_xor_sync(0xffffffffu, l, msk);
    if (lig == 0) {
      s_m[part][g] = m_run[g];
      s_l[part][g] = l;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) s_o[part][g][lig * 8 + e] = acc[g][e];
  }
  __syncthreads();
  const size_t pidx = static_cast<size_t>(S.part_base + chunk);
  for (int idx = threadIdx.x; idx < G * D_HEAD; idx += AT_THREADS) {
    const int g = idx / D_HEAD, c = idx % D_HEAD;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int pp = 0; pp < NPART; ++pp) M = fmaxf(M, s_m[pp][g]);
    const float Mu = (M == -CUDART_INF_F) ? 0.f : M;
    float o = 0.f, l = 0.f;
#pragma unroll
    for (int pp = 0; pp < NPART; ++pp) {
      const float w = exp2f(s_m[pp][g] - Mu);
      o = fmaf(w, s_o[pp][g][c], o);
      l = fmaf(w, s_l[pp][g], l);
    }
    const size_t hq = pidx * P.n_q + kvh * G + g;
    P.part_o[hq * D_HEAD + c] = o;
    if (c == 0) {
      P.part_ml[hq * 2] = M;
      P.part_ml[hq * 2 + 1] = l;
    }
  }
}

// Merge the chunk partials of one (sequence, query head) in chunk order and normalise.
template <int D_HEAD>
__global__ void __launch_bounds__(D_HEAD) kvd_attn_merge_kernel(const __grid_constant__ AttnLaunch P) {
  const int h = blockIdx.x;
  const int si = blockIdx.y;
  const AttnSeq &S = P.seq[si];
  const int c = threadIdx.x;
  float M = -CUDART_INF_F;
  for (int ch = 0; ch < S.n_chunks; ++ch)
    M = fmaxf(M, P.part_ml[(static_cast<size_t>(S.part_base + ch) * P.n_q + h) * 2]);
  const float Mu = (M == -CUDART_INF_F) ? 0.f : M;
  float o = 0.f, l = 0.f;
  for (int ch = 0; ch < S.n_chunks; ++ch) {
    const size_t hq = static_cast<size_t>(S.part_base + ch) * P.n_q + h;
    const float w = exp2f(P.part_ml[hq * 2] - Mu);
    o = fmaf(w, P.part_o[hq * D_HEAD + c], o);
    l = fmaf(w, P.part_ml[hq * 2 + 1], l);
  }
  const float r = l > 0.f ? o / l : 0.f;
  P.out[(static_cast<size_t>(si) * P.n_q + h) * D_HEAD + c] = __float2bfloat16_rn(r);
}

template <int D_HEAD, int G>
static kvd_status launch_attn_impl(kvd_ctx *ctx, const AttnLaunch &L, cudaStream_t stream) {
  if (L.total_chunks > 0) {
    dim3 grid(L.total_chunks, L.n_kv);
    kvd_attn_split_kernel<D_HEAD, G><<<grid, AT_THREADS, 0, stream>>>(L);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch attention split");
    ctx->launches += 1;
  }
  dim3 mgrid(L.n_q, L.n_seqs);
  kvd_attn_merge_kernel<D_HEAD><<<mgrid, D_HEAD, 0, stream>>>(L);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch attention merge");
  ctx->launches += 1;
  return KVD_OK;
}

template <int D_HEAD>
static kvd_status launch_attn_group(kvd_ctx *ctx, const AttnLaunch &L, int group, cudaStream_t stream) {
  switch (group) {
    case 1: return launch_attn_impl<D_HEAD, 1>(ctx, L, stream);
    case 2: return launch_attn_impl<D_HEAD, 2>(ctx, L, stream);
    case 3: return launch_attn_impl<D_HEAD, 3>(ctx, L, stream);
    case 4: return launch_attn_impl<D_HEAD, 4>(ctx, L, stream);
    case 8: return launch_attn_impl<D_HEAD, 8>(ctx, L, stream);
    default: return KVD_ERR_SHAPE;
  }
}

kvd_status launch_attention(kvd_ctx *ctx, const AttnLaunch &L, int d_head, int group, cudaStream_t stream) {
  switch (d_head) {
    case 64: return launch_attn_group<64>(ctx, L, group, stream);
    case 128: return launch_attn_group<128>(ctx, L, group, stream);
    case 256: return launch_attn_group<256>(ctx, L, group, stream);
    default: return KVD_ERR_SHAPE;
  }
}

}  // namespace kvd
