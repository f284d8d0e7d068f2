// Decode attention (paper Eq. 6-7; ATTENTION(Q, K_all, V_all) of Algorithm 1) for one query token
// per sequence, grouped-query heads, keys given as up to four position-contiguous segments.
//
// Split over keys: the visible position range of a sequence is cut into chunks aligned to absolute
// position.  One CTA handles one (chunk, KV head): it streams that head's K and V rows with
// coalesced 16-byte loads, every lane owning 8 channels, and serves all query heads of the group
// from the same loads.  Scores of 8 keys at a time are reduced across the lanes of a key with a
// transposing shuffle butterfly, the softmax runs online in base 2, and each CTA writes one partial
// (max, sum, unnormalised output) per query head.  A second, small kernel merges each head group's
// partials in chunk order and writes the output.  Streaming CTAs are four warps, four per SM: the
// CTAs of an SM overlap each other's start-up and combine phases, which matters in batched launches
// of many waves.
//
// Which chunk, warp, lane group and slot a key lands in is a function of its position only, and the
// merge runs in chunk order, so the output bits do not depend on how the keys are spread over
// segments.
#include <math_constants.h>
#include <string.h>

#include <atomic>

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

// DT: element type of q, K, V and the output (0 = bf16, 1 = fp16; kvd_set_dtype).
// ALLIN: for launches of at most two CTAs per SM whose chunks are two iterations long (a single sequence of
// a few thousand keys), where nothing else on the SM hides a load's latency: the loads of both iterations are
// issued before the query is fetched and before anything is computed, so a CTA pays one memory round trip
// instead of three.  The arithmetic and its order are the same, hence the same bits.
template <int D_HEAD, int G, int NSEQ, int DT = 0, bool ALLIN = false>
__global__ void __launch_bounds__(AT_THREADS, ALLIN ? 2 : AT_CTAS_PER_SM) kvd_attn_split_kernel(const __grid_constant__ AttnLaunchT<NSEQ> P) {
  constexpr int LPK = D_HEAD / 8;         // lanes per key
  constexpr int KPL = 32 / LPK;           // keys per warp-wide load
  constexpr int U = AT_UNROLL;            // keys per lane group per iteration
  constexpr int NPART = AT_WARPS * KPL;   // lane groups per CTA
  // The merge kernel is launched as a programmatic dependent of this one: once every CTA of this
  // grid has started, its CTAs may take SMs that become free and wait there (griddepcontrol.wait)
  // for this grid to complete, so its launch latency is off the critical path.
  grid_launch_dependents();
  // per lane group: unnormalised output, maximum, sum (AttnSmem<D_HEAD, G>::BYTES of dynamic shared memory)
  extern __shared__ __align__(16) float at_smem[];
  float (*s_o)[G][D_HEAD] = reinterpret_cast<float (*)[G][D_HEAD]>(at_smem);
  float (*s_m)[G] = reinterpret_cast<float (*)[G]>(at_smem + NPART * G * D_HEAD);
  float (*s_l)[G] = s_m + NPART;

  // ---- which (sequence, chunk) is this CTA's?
  int si = 0;
  {
    int lo = 0, hi = P.n_seqs - 1;
    const int b = blockIdx.x / P.n_kv;
    while (lo < hi) {  // last sequence whose first partial index is <= b
      const int mid = (lo + hi + 1) >> 1;
      if (P.seq[mid].part_base - P.seq[0].part_base <= b) lo = mid; else hi = mid - 1;
    }
    si = lo;
  }
  const AttnSeq &S = P.seq[si];
  const int chunk = blockIdx.x / P.n_kv - (S.part_base - P.seq[0].part_base);
  const int kvh = blockIdx.x % P.n_kv;  // the KV heads of one chunk are neighbours in the grid and in memory
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int grp = lane / LPK;   // lane group inside the warp
  const int lig = lane % LPK;   // lane inside the group: owns channels [8*lig, 8*lig + 8)
  const int my_slot = ((lig & (LPK / 2)) ? 4 : 0) + ((lig & (LPK / 4)) ? 2 : 0) + ((lig & (LPK / 8)) ? 1 : 0);
  const int chunk_keys = KPL * U * AT_WARPS * S.iters;
  const int chunk_pos0 = S.chunk0_pos + chunk * chunk_keys;

  // everything above used kernel parameters only; K, V and q may come from the preceding kernel
  grid_dependency_wait();
  // ---- query of every head of the group, pre-multiplied by scale * log2(e)
  uint64_t qf[G][4];  // channel pairs (2j, 2j+1)
  auto load_query = [&]() {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const __nv_bfloat16 *qp = P.q + (static_cast<size_t>(si) * P.n_q + kvh * G + g) * D_HEAD + lig * 8;
      const uint4 w = *reinterpret_cast<const uint4 *>(qp);
      const uint64_t sc2 = pack2(P.scale_log2e, P.scale_log2e);
      qf[g][0] = fmul2(x2_to_f32x2<DT>(w.x), sc2);
      qf[g][1] = fmul2(x2_to_f32x2<DT>(w.y), sc2);
      qf[g][2] = fmul2(x2_to_f32x2<DT>(w.z), sc2);
      qf[g][3] = fmul2(x2_to_f32x2<DT>(w.w), sc2);
    }
  };
  if constexpr (!ALLIN) load_query();

  float m_run[G], l_run[G];
  uint64_t acc[G][4];  // channel pairs
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m_run[g] = -CUDART_INF_F;
    l_run[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[g][e] = 0ull;
  }

  const size_t head_off = static_cast<size_t>(kvh) * D_HEAD + lig * 8;

  // Whole chunk inside one segment and inside the visible range (the common case): addresses are
  // linear in the position.  Otherwise every key is looked up in the segment list.  The choice is
  // uniform over the CTA and does not change which keys are read or in which order.
  int fast_seg = -1;
#pragma unroll
  for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg)
    if (chunk_pos0 >= S.first[sg] && chunk_pos0 + chunk_keys <= S.first[sg] + S.len[sg]) fast_seg = sg;
  const bool fast = fast_seg >= 0 && chunk_pos0 >= S.lo_pos && chunk_pos0 + chunk_keys - 1 <= S.hi_pos;
  const __nv_bfloat16 *fk = P.q, *fv = P.q;
  long long fstride = 0;
  if (fast) {
    fstride = S.stride[fast_seg];
    const size_t off = static_cast<size_t>(chunk_pos0 - S.first[fast_seg]) * fstride + head_off;
    fk = S.k[fast_seg] + off;
    fv = S.v[fast_seg] + off;
  }

  // issue the 16 loads of one iteration (8 keys, 8 values) for this lane group
  auto issue = [&](int it, uint4 (&kr)[U], uint4 (&vr)[U], uint32_t &vmask) {
    const int rel0 = ((it * AT_WARPS + warp) * KPL + grp) * U;  // first of this group's 8 positions
    if (fast) {
      const __nv_bfloat16 *kp = fk + static_cast<size_t>(rel0) * fstride;
      const __nv_bfloat16 *vp = fv + static_cast<size_t>(rel0) * fstride;
#pragma unroll
      for (int u = 0; u < U; ++u) kr[u] = ldg_stream(kp + u * fstride);
#pragma unroll
      for (int u = 0; u < U; ++u) vr[u] = ldg_stream(vp + u * fstride);
      vmask = 0xFFu;
    } else {
      // masked keys are not loaded: they read as zeros and score -inf
      vmask = 0;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int pos = chunk_pos0 + rel0 + u;
        const __nv_bfloat16 *kp = nullptr, *vp = nullptr;
        if (pos >= S.lo_pos && pos <= S.hi_pos) {
#pragma unroll
          for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
            const int r = pos - S.first[sg];
            if (r >= 0 && r < S.len[sg]) {
              const size_t off = static_cast<size_t>(r) * S.stride[sg] + head_off;
              kp = S.k[sg] + off;
              vp = S.v[sg] + off;
              vmask |= 1u << u;
            }
          }
        }
        kr[u] = make_uint4(0u, 0u, 0u, 0u);
        vr[u] = make_uint4(0u, 0u, 0u, 0u);
        if (kp != nullptr) {
          kr[u] = ldg_stream(kp);
          vr[u] = ldg_stream(vp);
        }
      }
    }
  };

  // scores, online softmax and weighted values for the 8 keys of one iteration
  auto compute = [&](const uint4 (&kr)[U], const uint4 (&vr)[U], uint32_t vmask) {
    // ---- scores: per-lane partial dot products (one key unpacked at a time), then the transposing
    // reduction
    float part[G][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint64_t k0 = x2_to_f32x2<DT>(kr[u].x), k1 = x2_to_f32x2<DT>(kr[u].y);
      const uint64_t k2 = x2_to_f32x2<DT>(kr[u].z), k3 = x2_to_f32x2<DT>(kr[u].w);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        // even and odd channels accumulate side by side, then are added
        uint64_t d = fmul2(qf[g][0], k0);
        d = ffma2(qf[g][1], k1, d);
        d = ffma2(qf[g][2], k2, d);
        d = ffma2(qf[g][3], k3, d);
        float de, dodd;
        unpack2(d, de, dodd);
        part[g][u] = de + dodd;
      }
    }
    float pb[G][U];  // softmax numerators of the 8 keys, broadcast to every lane of the group
    float corr[G];
    const bool my_valid = (vmask >> my_slot) & 1u;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float sc = reduce8_transposed<LPK>(part[g], lig);
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
        const int srcl = grp * LPK + ((u & 4) ? LPK / 2 : 0) + ((u & 2) ? LPK / 4 : 0) + ((u & 1) ? LPK / 8 : 0);
        pb[g][u] = __shfl_sync(0xffffffffu, pmine, srcl);
      }
    }
    // ---- weighted values
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint64_t c2 = pack2(corr[g], corr[g]);
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[g][e] = fmul2(acc[g][e], c2);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint64_t v0 = x2_to_f32x2<DT>(vr[u].x), v1 = x2_to_f32x2<DT>(vr[u].y);
      const uint64_t v2 = x2_to_f32x2<DT>(vr[u].z), v3 = x2_to_f32x2<DT>(vr[u].w);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const uint64_t p2 = pack2(pb[g][u], pb[g][u]);
        acc[g][0] = ffma2(p2, v0, acc[g][0]);
        acc[g][1] = ffma2(p2, v1, acc[g][1]);
        acc[g][2] = ffma2(p2, v2, acc[g][2]);
        acc[g][3] = ffma2(p2, v3, acc[g][3]);
      }
    }
  };
  // a warp none of whose keys is visible has nothing to add (warp-uniform test: the reductions
  // inside compute() use the whole warp)
  auto step = [&](const uint4 (&kr)[U], const uint4 (&vr)[U], uint32_t vmask) {
    if (__any_sync(0xffffffffu, vmask != 0u)) compute(kr, vr, vmask);
  };

  if constexpr (ALLIN) {
    // both iterations' loads, then the query, then the arithmetic in the usual order
    uint4 ka[U], va[U], kb[U], vb[U];
    uint32_t ma = 0, mb = 0;
    issue(0, ka, va, ma);
    issue(1, kb, vb, mb);
    load_query();
    step(ka, va, ma);
    step(kb, vb, mb);
  } else {
    // One buffer of loads per iteration; latency is hidden by the other 15 warps resident on the SM
    // (the kernel is capped at 128 registers so that four CTAs fit), which measured faster than
    // register double buffering or a shared-memory ring at half the occupancy.
    uint4 ka[U], va[U];
    uint32_t ma = 0;
    for (int it = 0; it < S.iters; ++it) {
      issue(it, ka, va, ma);
      step(ka, va, ma);
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
    for (int e = 0; e < 4; ++e) {
      float a0, a1;
      unpack2(acc[g][e], a0, a1);
      s_o[part][g][lig * 8 + 2 * e] = a0;
      s_o[part][g][lig * 8 + 2 * e + 1] = a1;
    }
  }
  __syncthreads();
  const size_t pidx = static_cast<size_t>(S.slot_base + chunk);
  for (int idx = threadIdx.x; idx < G * D_HEAD; idx += AT_THREADS) {
    const int g = idx / D_HEAD, c = idx % D_HEAD;
    float M = -CUDART_INF_F;
#pragma unroll 8
    for (int pp = 0; pp < NPART; ++pp) M = fmaxf(M, s_m[pp][g]);
    const float Mu = (M == -CUDART_INF_F) ? 0.f : M;
    float o = 0.f, l = 0.f;
#pragma unroll 8
    for (int pp = 0; pp < NPART; ++pp) {
      const float w = exp2f(s_m[pp][g] - Mu);
      o = fmaf(w, s_o[pp][g][c], o);
      l = fmaf(w, s_l[pp][g], l);
    }
    const size_t hq = pidx * P.n_q + kvh * G + g;
    if (!KVD_BOUNDS_OK(pidx < static_cast<size_t>(P.max_parts), P.status)) continue;  // checking build: the partial's slot
    P.part_o[hq * D_HEAD + c] = o;
    if (c == 0) {
      P.part_ml[hq * 2] = M;
      P.part_ml[hq * 2 + 1] = l;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Streaming kernel for wide query groups (G >= 3, d_head <= 128).  With four or more query heads per
// KV head the fp32 pipes, not the loads, bound the kernel above (about 45 warp instructions per key),
// so the two products run on the tensor cores with the query heads padded to a 16-row tile:
//     S (16 heads x 8 keys)         = Q (16 x d_head) * K^T            mma.m16n8k16, d_head/16 per 8 keys
//     O^T (d_head x 8 heads)       += V^T (d_head x 8 keys) * P^T      mma.m16n8k8,  d_head/16 per 8 keys
// Operands come straight from global memory with the same 16-byte loads: a contraction does not care
// which channel (or key) sits in which slot as long as both operands agree, so each thread loads
// contiguous 16-byte pieces and uses them as the fragment registers the instruction wants -- K pieces
// as B fragments of the first product (the query is loaded the same way), pairs of V pieces of two
// neighbouring keys, interleaved with two byte permutes, as A fragments of the second.  P is rounded
// to bf16 for the second product (fp32 sums), as the scores' softmax weights are in any tensor-core
// attention; the partials have the same format as those of the kernel above and go to the same merge.
// Chunking, the position -> (chunk, warp, block) assignment and the masking rules are identical.
template <int DT>
__device__ __forceinline__ void mma_x16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  if constexpr (DT == 0)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  else
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <int DT>
__device__ __forceinline__ void mma_x16_m16n8k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  if constexpr (DT == 0)
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(b0));
  else
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(b0));
}

template <int D_HEAD, int G, int NSEQ, int DT = 0>
__global__ void __launch_bounds__(AT_THREADS, AT_CTAS_PER_SM)
    kvd_attn_split_mma_kernel(const __grid_constant__ AttnLaunchT<NSEQ> P) {
  static_assert(G >= 1 && G <= 8 && D_HEAD <= 128, "query heads are the 8 columns of the second product");
  constexpr int LPK = D_HEAD / 8, KPL = 32 / LPK;
  constexpr int WARP_KEYS = KPL * AT_UNROLL;  // keys per warp and iteration, as in the kernel above
  constexpr int NBLK = WARP_KEYS / 8;         // blocks of 8 keys
  constexpr int KP = D_HEAD / 32;             // 16-byte pieces of a key row per thread (first product)
  constexpr int VP = D_HEAD / 64;             // 16-byte pieces of a value row per thread (second product)
  constexpr int MB = D_HEAD / 16;             // 16-channel blocks of the output
  __shared__ float s_o[AT_WARPS][G][D_HEAD];
  __shared__ float s_m[AT_WARPS][G];
  __shared__ float s_l[AT_WARPS][G];
  grid_launch_dependents();

  int si = 0;
  {
    int lo = 0, hi = P.n_seqs - 1;
    const int b = blockIdx.x / P.n_kv;
    while (lo < hi) {  // last sequence whose first partial index is <= b
      const int mid = (lo + hi + 1) >> 1;
      if (P.seq[mid].part_base - P.seq[0].part_base <= b) lo = mid; else hi = mid - 1;
    }
    si = lo;
  }
  const AttnSeq &S = P.seq[si];
  const int chunk = blockIdx.x / P.n_kv - (S.part_base - P.seq[0].part_base);
  const int kvh = blockIdx.x % P.n_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2;  // fragment row / column index: query head, key of a block, channel group
  const int t = lane & 3;    // fragment pair index
  const int chunk_keys = WARP_KEYS * AT_WARPS * S.iters;
  const int chunk_pos0 = S.chunk0_pos + chunk * chunk_keys;

  grid_dependency_wait();
  // ---- query rows as A fragments: thread (g8, t) holds channels [32 j + 8 t, 32 j + 8 t + 8) of head g8
  uint32_t qa[KP][4];
#pragma unroll
  for (int j = 0; j < KP; ++j) {
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (g8 < G)
      w = *reinterpret_cast<const uint4 *>(P.q + (static_cast<size_t>(si) * P.n_q + kvh * G + g8) * D_HEAD + 32 * j + 8 * t);
    qa[j][0] = w.x;
    qa[j][1] = w.y;
    qa[j][2] = w.z;
    qa[j][3] = w.w;
  }
  float m_run = -CUDART_INF_F, l_run = 0.f;  // of head g8 (threads with g8 >= G carry padding)
  float oacc[MB][4];                         // O^T: rows = channels of this thread's group, columns = heads 2t, 2t+1
#pragma unroll
  for (int mb = 0; mb < MB; ++mb)
#pragma unroll
    for (int r = 0; r < 4; ++r) oacc[mb][r] = 0.f;

  const size_t head_el = static_cast<size_t>(kvh) * D_HEAD;
  int fast_seg = -1;
#pragma unroll
  for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg)
    if (chunk_pos0 >= S.first[sg] && chunk_pos0 + chunk_keys <= S.first[sg] + S.len[sg]) fast_seg = sg;
  const bool fast = fast_seg >= 0 && chunk_pos0 >= S.lo_pos && chunk_pos0 + chunk_keys - 1 <= S.hi_pos;
  const __nv_bfloat16 *fk = P.q, *fv = P.q;
  long long fstride = 0;
  if (fast) {
    fstride = S.stride[fast_seg];
    const size_t off = static_cast<size_t>(chunk_pos0 - S.first[fast_seg]) * fstride + head_el;
    fk = S.k[fast_seg] + off;
    fv = S.v[fast_seg] + off;
  }
  // row pointers (K, V) of the key at chunk-relative position rel, or null when it is not visible
  auto locate = [&](int rel, const __nv_bfloat16 *&kp, const __nv_bfloat16 *&vp) {
    kp = vp = nullptr;
    if (fast) {
      kp = fk + static_cast<size_t>(rel) * fstride;
      vp = fv + static_cast<size_t>(rel) * fstride;
      return;
    }
    const int pos = chunk_pos0 + rel;
    if (pos >= S.lo_pos && pos <= S.hi_pos) {
#pragma unroll
      for (int sg = 0; sg < KVD_MAX_SEGMENTS; ++sg) {
        const int r = pos - S.first[sg];
        if (r >= 0 && r < S.len[sg]) {
          const size_t off = static_cast<size_t>(r) * S.stride[sg] + head_el;
          kp = S.k[sg] + off;
          vp = S.v[sg] + off;
        }
      }
    }
  };

  for (int it = 0; it < S.iters; ++it) {
    const int rel0 = (it * AT_WARPS + warp) * WARP_KEYS;
    // ---- all loads of the iteration: per block, the key row of key g8 (first product) and the value
    // rows of keys 2t and 2t+1 (second product); invisible keys read as zeros
    uint4 kr[NBLK][KP], vr[NBLK][2][VP];
    uint32_t vmask = 0;  // bit 2b + i: key 8b + 2t + i is visible
#pragma unroll
    for (int b = 0; b < NBLK; ++b) {
      const __nv_bfloat16 *kp, *vp_unused, *kp_unused, *vp0, *vp1;
      locate(rel0 + 8 * b + g8, kp, vp_unused);
      locate(rel0 + 8 * b + 2 * t, kp_unused, vp0);
      locate(rel0 + 8 * b + 2 * t + 1, kp_unused, vp1);
#pragma unroll
      for (int j = 0; j < KP; ++j)
        kr[b][j] = kp ? ldg_stream(kp + 32 * j + 8 * t) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int i = 0; i < VP; ++i) {
        vr[b][0][i] = vp0 ? ldg_stream(vp0 + 64 * i + 8 * g8) : make_uint4(0u, 0u, 0u, 0u);
        vr[b][1][i] = vp1 ? ldg_stream(vp1 + 64 * i + 8 * g8) : make_uint4(0u, 0u, 0u, 0u);
      }
      vmask |= (vp0 ? 1u : 0u) << (2 * b);
      vmask |= (vp1 ? 1u : 0u) << (2 * b + 1);
    }
    if (!__any_sync(0xffffffffu, vmask != 0u)) continue;  // nothing visible in this warp's keys

#pragma unroll
    for (int b = 0; b < NBLK; ++b) {
      // ---- scores of 8 keys for (up to) 8 heads
      float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KP; ++j) {
        mma_x16_m16n8k16<DT>(sc, qa[j][0], 0u, qa[j][1], 0u, kr[b][j].x, kr[b][j].y);
        mma_x16_m16n8k16<DT>(sc, qa[j][2], 0u, qa[j][3], 0u, kr[b][j].z, kr[b][j].w);
      }
      // thread (g8, t): head g8, keys 2t and 2t+1 of the block
      const float s0 = ((vmask >> (2 * b)) & 1u) ? sc[0] * P.scale_log2e : -CUDART_INF_F;
      const float s1 = ((vmask >> (2 * b + 1)) & 1u) ? sc[1] * P.scale_log2e : -CUDART_INF_F;
      float bmax = fmaxf(s0, s1);
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
      const float m_new = fmaxf(m_run, bmax);
      const float m_use = (m_new == -CUDART_INF_F) ? 0.f : m_new;
      const float corr = exp2f(m_run - m_use);  // 0 while nothing has been seen
      const float p0 = exp2f(s0 - m_use), p1 = exp2f(s1 - m_use);
      l_run = fmaf(l_run, corr, p0 + p1);
      m_run = m_new;
      const uint32_t pk = pack_out<DT>(p0, p1);  // B fragment of the second product: keys 2t, 2t+1, head g8
      // ---- rescale the accumulators when a maximum moved (columns are heads 2t and 2t+1)
      const float c_even = __shfl_sync(0xffffffffu, corr, (2 * t) * 4);
      const float c_odd = __shfl_sync(0xffffffffu, corr, (2 * t + 1) * 4);
      if (__any_sync(0xffffffffu, c_even != 1.0f || c_odd != 1.0f)) {
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          oacc[mb][0] *= c_even;
          oacc[mb][1] *= c_odd;
          oacc[mb][2] *= c_even;
          oacc[mb][3] *= c_odd;
        }
      }
      // ---- weighted values: A fragment rows are this thread's channels 64 i + 8 g8 + 2 e (+1), taken
      // from keys 2t (low half) and 2t+1 (high half)
#pragma unroll
      for (int i = 0; i < VP; ++i) {
        const uint32_t v0[4] = {vr[b][0][i].x, vr[b][0][i].y, vr[b][0][i].z, vr[b][0][i].w};
        const uint32_t v1[4] = {vr[b][1][i].x, vr[b][1][i].y, vr[b][1][i].z, vr[b][1][i].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t a0 = __byte_perm(v0[e], v1[e], 0x5410);  // channel 2e of both keys
          const uint32_t a1 = __byte_perm(v0[e], v1[e], 0x7632);  // channel 2e + 1 of both keys
          mma_x16_m16n8k8<DT>(oacc[4 * i + e], a0, a1, pk);
        }
      }
    }
  }

  // ---- one partial per warp into shared memory, then the CTA's partial as in the kernel above
  {
    float l = l_run;
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (t == 0 && g8 < G) {
      s_m[warp][g8] = m_run;
      s_l[warp][g8] = l;
    }
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) {
      const int ch = 64 * (mb >> 2) + 8 * g8 + 2 * (mb & 3);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int head = 2 * t + (r & 1);
        if (head < G) s_o[warp][head][ch + (r >> 1)] = oacc[mb][r];
      }
    }
  }
  __syncthreads();
  const size_t pidx = static_cast<size_t>(S.slot_base + chunk);
  for (int idx = threadIdx.x; idx < G * D_HEAD; idx += AT_THREADS) {
    const int g = idx / D_HEAD, c = idx % D_HEAD;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int pp = 0; pp < AT_WARPS; ++pp) M = fmaxf(M, s_m[pp][g]);
    const float Mu = (M == -CUDART_INF_F) ? 0.f : M;
    float o = 0.f, l = 0.f;
#pragma unroll
    for (int pp = 0; pp < AT_WARPS; ++pp) {
      const float w = exp2f(s_m[pp][g] - Mu);
      o = fmaf(w, s_o[pp][g][c], o);
      l = fmaf(w, s_l[pp][g], l);
    }
    const size_t hq = pidx * P.n_q + kvh * G + g;
    if (!KVD_BOUNDS_OK(pidx < static_cast<size_t>(P.max_parts), P.status)) continue;  // checking build: the partial's slot
    P.part_o[hq * D_HEAD + c] = o;
    if (c == 0) {
      P.part_ml[hq * 2] = M;
      P.part_ml[hq * 2 + 1] = l;
    }
  }
}

// Second kernel of a decode step: the chunk partials of every (sequence, KV head) are merged in chunk
// order and the output written.  A separate launch instead of a "last CTA merges" tail: every
// dependent global-memory hop (partial -> fence -> counter -> merge) measured above a microsecond,
// which the streaming CTAs would spend idle on their SM; the kernel boundary costs about as much
// once per step and needs no counters.  A sequence without a visible key gets zeros.
//
// One CTA per (sequence, KV head, slice of 64 channels).  Warp w merges the w-th group of consecutive
// partials of its head group, each lane owning two channels of every head: a partial costs a lane 4*G
// registers, a group is as many partials as fit 64 registers (attn_merge_group(G)), all fetched at
// once, so a warp's work is one round trip to the L2; the warp results are added in warp order.  The
// launch has as many warps per CTA as its longest sequence has groups (at most 16; beyond that a warp
// takes several groups, 16 apart); a shorter sequence leaves the extra warps idle, so its summation
// order depends on its own chunk count only.
template <int D_HEAD, int G, int NSEQ, int DT = 0>
__global__ void __launch_bounds__(AT_MERGE_THREADS)
    kvd_attn_merge_kernel(const __grid_constant__ AttnLaunchT<NSEQ> P) {
  constexpr int SLICES = D_HEAD / AT_MERGE_SLICE;
  constexpr int PF = attn_merge_group(G);
  __shared__ float s_o[AT_MERGE_WARPS][G][AT_MERGE_SLICE];
  __shared__ float s_l[AT_MERGE_WARPS][G];
  const int slice = blockIdx.x % SLICES;
  const int head_slot = blockIdx.x / SLICES;
  const int si = head_slot / P.n_kv, kvh = head_slot % P.n_kv;
  const AttnSeq &S = P.seq[si];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  grid_launch_dependents();
  // wait until the preceding grid in the stream (the streaming kernel) has completed and its
  // partials are visible
  grid_dependency_wait();

  // (checking build: the slots to merge lie inside the partial arrays; otherwise nothing is merged)
  const int count = KVD_BOUNDS_OK(S.merge_base >= 0 && S.merge_base + S.merge_count <= P.max_parts, P.status) ? S.merge_count : 0;
  const int n_groups = (count + PF - 1) / PF;
  const int warps_used = n_groups < AT_MERGE_WARPS ? n_groups : AT_MERGE_WARPS;
  const float *ml0 = P.part_ml + (static_cast<size_t>(S.merge_base) * P.n_q + kvh * G) * 2;
  const float *po0 = P.part_o + (static_cast<size_t>(S.merge_base) * P.n_q + kvh * G) * D_HEAD +
                     slice * AT_MERGE_SLICE + lane * 2;
  const size_t ml_stride = static_cast<size_t>(P.n_q) * 2, po_stride = static_cast<size_t>(P.n_q) * D_HEAD;
  if (warp < warps_used) {
    float2 vbuf[PF][G], mlbuf[PF][G];
    // (a partial past the end re-reads the last one and is skipped below: no branch between the loads)
    auto fetch_group = [&](int grp) {
#pragma unroll
      for (int i = 0; i < PF; ++i) {
        const int ch = grp * PF + i < count ? grp * PF + i : count - 1;
#pragma unroll
        for (int g = 0; g < G; ++g) {
          mlbuf[i][g] = __ldcg(reinterpret_cast<const float2 *>(ml0 + ch * ml_stride + g * 2));
          vbuf[i][g] = __ldcg(reinterpret_cast<const float2 *>(po0 + ch * po_stride + g * D_HEAD));
        }
      }
    };
    fetch_group(warp);
    // the maximum of each head over all partials: lanes over partials (the first 256 loaded before
    // any is used), then shuffles -- every warp by itself, no block barrier
    float Mu[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float mv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int ch = lane + 32 * i;
        mv[i] = ch < count ? __ldcg(ml0 + ch * ml_stride + g * 2) : -CUDART_INF_F;
      }
      float mx = fmaxf(fmaxf(fmaxf(mv[0], mv[1]), fmaxf(mv[2], mv[3])), fmaxf(fmaxf(mv[4], mv[5]), fmaxf(mv[6], mv[7])));
      for (int ch = lane + 256; ch < count; ch += 32) mx = fmaxf(mx, __ldcg(ml0 + ch * ml_stride + g * 2));
#pragma unroll
      for (int msk = 16; msk >= 1; msk >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, msk));
      Mu[g] = (mx == -CUDART_INF_F) ? 0.f : mx;
    }
    float2 o[G];
    float l[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      l[g] = 0.f;
      o[g] = make_float2(0.f, 0.f);
    }
    for (int grp = warp; grp < n_groups; grp += AT_MERGE_WARPS) {
      if (grp != warp) fetch_group(grp);
#pragma unroll
      for (int i = 0; i < PF; ++i) {
        if (grp * PF + i < count) {
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float w = exp2f(mlbuf[i][g].x - Mu[g]);
            l[g] = fmaf(w, mlbuf[i][g].y, l[g]);
            o[g].x = fmaf(w, vbuf[i][g].x, o[g].x);
            o[g].y = fmaf(w, vbuf[i][g].y, o[g].y);
          }
        }
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (lane == 0) s_l[warp][g] = l[g];
      s_o[warp][g][lane * 2] = o[g].x;
      s_o[warp][g][lane * 2 + 1] = o[g].y;
    }
  }
  __syncthreads();
  // the warp sums are added in warp order
  for (int idx = threadIdx.x; idx < G * AT_MERGE_SLICE; idx += blockDim.x) {
    const int g = idx / AT_MERGE_SLICE, c = idx % AT_MERGE_SLICE;
    float ov = 0.f, lv = 0.f;
    for (int w = 0; w < warps_used; ++w) {
      ov += s_o[w][g][c];
      lv += s_l[w][g];
    }
    const float r = lv > 0.f ? ov / lv : 0.f;
    const size_t oi = (static_cast<size_t>(si) * P.n_q + kvh * G + g) * D_HEAD + slice * AT_MERGE_SLICE + c;
    if constexpr (DT == 0) P.out[oi] = __float2bfloat16_rn(r);
    else reinterpret_cast<__half *>(P.out)[oi] = __float2half_rn(r);
  }
}

// dynamic shared memory of the kernel and its one-time opt-in (sizes above 48 KB need it)
template <int D_HEAD, int G>
struct AttnSmem {
  static constexpr int NPART = AT_WARPS * (32 / (D_HEAD / 8));
  static constexpr int BYTES = NPART * G * (D_HEAD + 2) * 4;
};
template <int D_HEAD, int G, int NSEQ, int DT>
static cudaError_t attn_configure() {
  static bool done[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!done[dev & 63]) {
    if constexpr (!(G >= 3 && D_HEAD <= 128)) {
      e = cudaFuncSetAttribute(kvd_attn_split_kernel<D_HEAD, G, NSEQ, DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               AttnSmem<D_HEAD, G>::BYTES);
      if (e != cudaSuccess) return e;
      if constexpr (G <= 2) {
        e = cudaFuncSetAttribute(kvd_attn_split_kernel<D_HEAD, G, NSEQ, DT, true>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<D_HEAD, G>::BYTES);
        if (e != cudaSuccess) return e;
      }
    }
    done[dev & 63] = true;
  }
  return cudaSuccess;
}
// the two launches of a decode step: stream + partials, then merge
template <int D_HEAD, int G, int NSEQ, int DT = 0>
static cudaError_t attn_launch_pair(const AttnLaunchT<NSEQ> &S, cudaStream_t stream) {
  cudaError_t e = attn_configure<D_HEAD, G, NSEQ, DT>();
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // Starting early pays for launches of up to one wave (the set-up hides under the predecessor's tail);
  // a many-wave grid whose first CTAs sit on the SMs waiting slowed a short predecessor down in
  // measurements (11 us lost on a 24 us predecessor), so those are ordered plainly.
  const bool small = S.total_chunks * S.n_kv <= 148 * AT_CTAS_PER_SM;
  if (S.total_chunks > 0) {
    attr[0].val.programmaticStreamSerializationAllowed = (small && !(serial_launch_mask() & 2)) ? 1 : 0;
    cfg.gridDim = dim3(S.total_chunks * S.n_kv, 1, 1);
    cfg.blockDim = dim3(AT_THREADS, 1, 1);
    if constexpr (G >= 3 && D_HEAD <= 128) {
      cfg.dynamicSmemBytes = 0;
      e = cudaLaunchKernelEx(&cfg, kvd_attn_split_mma_kernel<D_HEAD, G, NSEQ, DT>, S);
    } else {
      cfg.dynamicSmemBytes = AttnSmem<D_HEAD, G>::BYTES;
      // at most two CTAs per SM, every chunk two iterations long: the variant that issues all loads at once
      bool allin = G <= 2 && S.total_chunks * S.n_kv <= 148 * 2;
      for (int i = 0; i < S.n_seqs; ++i) allin = allin && (S.seq[i].n_chunks == 0 || S.seq[i].iters == 2);
      if constexpr (G <= 2) {
        if (allin) e = cudaLaunchKernelEx(&cfg, kvd_attn_split_kernel<D_HEAD, G, NSEQ, DT, true>, S);
        else e = cudaLaunchKernelEx(&cfg, kvd_attn_split_kernel<D_HEAD, G, NSEQ, DT>, S);
      } else {
        e = cudaLaunchKernelEx(&cfg, kvd_attn_split_kernel<D_HEAD, G, NSEQ, DT>, S);
      }
    }
    if (e != cudaSuccess) return e;
  }
  attr[0].val.programmaticStreamSerializationAllowed = (small && !(serial_launch_mask() & 4)) ? 1 : 0;
  // as many warps per merge CTA as the longest sequence of the launch has groups of partials
  int max_chunks = 1;
  for (int i = 0; i < S.n_seqs; ++i) max_chunks = S.seq[i].merge_count > max_chunks ? S.seq[i].merge_count : max_chunks;
  int merge_warps = (max_chunks + attn_merge_group(G) - 1) / attn_merge_group(G);
  if (merge_warps > AT_MERGE_WARPS) merge_warps = AT_MERGE_WARPS;
  cfg.gridDim = dim3(S.n_seqs * S.n_kv * (D_HEAD / AT_MERGE_SLICE), 1, 1);
  cfg.blockDim = dim3(32 * merge_warps, 1, 1);
  cfg.dynamicSmemBytes = 0;
  return cudaLaunchKernelEx(&cfg, kvd_attn_merge_kernel<D_HEAD, G, NSEQ, DT>, S);
}

template <int D_HEAD, int G, int NSEQ>
static kvd_status launch_attn_impl(kvd_ctx *ctx, const AttnLaunch &L, cudaStream_t stream) {
  if (L.n_seqs > 0) {
    static thread_local AttnLaunchT<NSEQ> S;
    static_cast<AttnLaunchHead &>(S) = static_cast<const AttnLaunchHead &>(L);
    for (int i = 0; i < L.n_seqs; ++i) S.seq[i] = L.seq[i];
    // fp16 contexts (kvd_set_dtype): the same kernels reading and writing fp16
    cudaError_t e = ctx->dtype == 1 ? attn_launch_pair<D_HEAD, G, NSEQ, 1>(S, stream)
                                    : attn_launch_pair<D_HEAD, G, NSEQ, 0>(S, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "launch attention");
    ctx->launches += L.total_chunks > 0 ? 2 : 1;
  }
  return KVD_OK;
}

template <int D_HEAD, int G>
static kvd_status launch_attn_nseq(kvd_ctx *ctx, const AttnLaunch &L, cudaStream_t stream) {
  if (L.n_seqs <= 4) return launch_attn_impl<D_HEAD, G, 4>(ctx, L, stream);
  return launch_attn_impl<D_HEAD, G, AT_MAX_SEQS>(ctx, L, stream);
}

template <int D_HEAD>
static kvd_status launch_attn_group(kvd_ctx *ctx, const AttnLaunch &L, int group, cudaStream_t stream) {
  switch (group) {
    case 1: return launch_attn_nseq<D_HEAD, 1>(ctx, L, stream);
    case 2: return launch_attn_nseq<D_HEAD, 2>(ctx, L, stream);
    case 3: return launch_attn_nseq<D_HEAD, 3>(ctx, L, stream);
    case 4: return launch_attn_nseq<D_HEAD, 4>(ctx, L, stream);
    case 8: return launch_attn_nseq<D_HEAD, 8>(ctx, L, stream);
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

// ------------------------------------------------------------------------------------------------
// kvd_decode_attention_static: decode attention for callers that cannot allocate device memory.
//
// The split partials live in the file-scope device array below instead of
// a caller-provided workspace.  Every GPU that loads this library holds the array until the process
// exits.  All calls share it, so two calls whose kernels overlap on one GPU race on it.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_kvd_static_scratch[KVD_STATIC_SCRATCH_BYTES];

namespace kvd {


// Device address of g_kvd_static_scratch on the current device.  The array's name is only a host-side
// handle; the address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
static kvd_status static_scratch_address(unsigned char **out) {
  static std::atomic<unsigned char *> cached[64] = {};  // host threads may make a device's first call together
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return KVD_ERR_UNSUPPORTED;
  }
  if (dev < 0 || dev >= 64) return KVD_ERR_UNSUPPORTED;
  if (cached[dev].load(std::memory_order_acquire) == nullptr) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_kvd_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return KVD_ERR_CUDA;
    }
    cached[dev].store(static_cast<unsigned char *>(p), std::memory_order_release);
  }
  *out = cached[dev].load(std::memory_order_acquire);
  return KVD_OK;
}

template <int D_HEAD, int G>
static kvd_status static_launch_g(const AttnLaunch &L, cudaStream_t stream) {
  static thread_local AttnLaunchT<AT_MAX_SEQS> S;
  static_cast<AttnLaunchHead &>(S) = static_cast<const AttnLaunchHead &>(L);
  for (int i = 0; i < L.n_seqs; ++i) S.seq[i] = L.seq[i];
  if (attn_launch_pair<D_HEAD, G, AT_MAX_SEQS>(S, stream) != cudaSuccess) {
    cudaGetLastError();
    return KVD_ERR_CUDA;
  }
  return KVD_OK;
}

template <int D_HEAD>
static kvd_status static_launch_d(const AttnLaunch &L, int group, cudaStream_t stream) {
  switch (group) {
    case 1: return static_launch_g<D_HEAD, 1>(L, stream);
    case 2: return static_launch_g<D_HEAD, 2>(L, stream);
    case 3: return static_launch_g<D_HEAD, 3>(L, stream);
    case 4: return static_launch_g<D_HEAD, 4>(L, stream);
    case 8: return static_launch_g<D_HEAD, 8>(L, stream);
    default: return KVD_ERR_SHAPE;
  }
}

}  // namespace kvd

extern "C" kvd_status kvd_decode_attention_static(int n_q_heads, int n_kv_heads, int d_head, int sliding_window,
                                                  int batch, const void *q, const int32_t *q_pos,
                                                  const kvd_kv_segment *segs, int n_segs, float scale, void *out,
                                                  void *stream_) {
  using namespace kvd;
  // ---- shapes and arguments (host only)
  if (n_q_heads <= 0 || n_kv_heads <= 0 || sliding_window < 0 || batch < 0 || n_segs < 0 ||
      n_segs > KVD_MAX_SEGMENTS)
    return KVD_ERR_INVALID_ARG;
  if (d_head != 64 && d_head != 128 && d_head != 256) return KVD_ERR_SHAPE;
  if (n_q_heads % n_kv_heads != 0) return KVD_ERR_SHAPE;
  const int group = n_q_heads / n_kv_heads;
  if (!(group == 1 || group == 2 || group == 3 || group == 4 || group == 8)) return KVD_ERR_SHAPE;
  if (batch == 0) return KVD_OK;
  if (!q || !q_pos || !out || (n_segs > 0 && !segs)) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return KVD_ERR_ALIGNMENT;
  // ---- limits of the fixed scratch: one launch pair, room for every partial
  if (batch > AT_MAX_SEQS) return KVD_ERR_CAPACITY;
  if (static_cast<size_t>(batch) * n_kv_heads > 1024) return KVD_ERR_CAPACITY;
  const int kdim = n_kv_heads * d_head;
  for (int b = 0; b < batch; ++b) {
    if (q_pos[b] < 0) return KVD_ERR_INVALID_ARG;
    for (int s = 0; s < n_segs; ++s) {
      const kvd_kv_segment &sg = segs[static_cast<size_t>(b) * n_segs + s];
      if (sg.len < 0 || sg.first_pos < 0) return KVD_ERR_INVALID_ARG;
      if (sg.len == 0) continue;
      if (!sg.k || !sg.v || sg.row_stride < kdim) return KVD_ERR_INVALID_ARG;
      if ((reinterpret_cast<uintptr_t>(sg.k) & 15u) || (reinterpret_cast<uintptr_t>(sg.v) & 15u) ||
          sg.row_stride % 8 != 0)
        return KVD_ERR_ALIGNMENT;
      if (static_cast<int64_t>(sg.first_pos) + sg.len > INT32_MAX) return KVD_ERR_INVALID_ARG;
      for (int s2 = 0; s2 < s; ++s2) {
        const kvd_kv_segment &o = segs[static_cast<size_t>(b) * n_segs + s2];
        if (o.len == 0) continue;
        if (sg.first_pos < o.first_pos + o.len && o.first_pos < sg.first_pos + sg.len) return KVD_ERR_INVALID_ARG;
      }
    }
  }
  // ---- the same position-based split as kvd_decode_attention
  static thread_local AttnLaunch L;
  int parts = 0;
  for (int b = 0; b < batch; ++b) {
    AttnSeq &S = L.seq[b];
    int min_first = INT32_MAX, max_last = -1;
    for (int s = 0; s < KVD_MAX_SEGMENTS; ++s) {
      S.k[s] = S.v[s] = nullptr;
      S.stride[s] = 0;
      S.first[s] = 0;
      S.len[s] = 0;
      if (s < n_segs) {
        const kvd_kv_segment &sg = segs[static_cast<size_t>(b) * n_segs + s];
        if (sg.len > 0) {
          S.k[s] = static_cast<const __nv_bfloat16 *>(sg.k);
          S.v[s] = static_cast<const __nv_bfloat16 *>(sg.v);
          S.stride[s] = sg.row_stride;
          S.first[s] = sg.first_pos;
          S.len[s] = sg.len;
          if (sg.first_pos < min_first) min_first = sg.first_pos;
          if (sg.first_pos + sg.len - 1 > max_last) max_last = sg.first_pos + sg.len - 1;
        }
      }
    }
    S.q_pos = q_pos[b];
    int lo = sliding_window > 0 ? S.q_pos - sliding_window + 1 : 0;
    if (lo < 0) lo = 0;
    if (min_first > lo) lo = min_first;
    const int hi = S.q_pos < max_last ? S.q_pos : max_last;
    S.lo_pos = lo;
    S.hi_pos = hi;
    S.part_base = parts;
    if (max_last < 0 || hi < lo) {
      S.n_chunks = 0;
      S.iters = 1;
      S.chunk0_pos = 0;
    } else {
      S.iters = attn_iters_for_span(d_head, n_kv_heads, hi - lo + 1);
      const int ck = attn_chunk_keys(d_head, S.iters);
      S.chunk0_pos = lo / ck * ck;
      S.n_chunks = hi / ck - lo / ck + 1;
    }
    S.slot_base = S.merge_base = S.part_base;
    S.merge_count = S.n_chunks;
    parts += S.n_chunks;
  }
  // one partial per chunk
  const size_t all_parts = static_cast<size_t>(parts);
  const size_t ml_bytes = (all_parts * n_q_heads * 2 * sizeof(float) + 255) / 256 * 256;
  const size_t o_bytes = all_parts * n_q_heads * d_head * sizeof(float);
  if (ml_bytes + o_bytes > static_cast<size_t>(KVD_STATIC_SCRATCH_BYTES)) return KVD_ERR_CAPACITY;

  unsigned char *scratch = nullptr;
  kvd_status st = static_scratch_address(&scratch);  // first call on a device: symbol look-up
  if (st != KVD_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  L.n_seqs = batch;
  L.total_chunks = parts;
  L.n_q = n_q_heads;
  L.n_kv = n_kv_heads;
  L.scale_log2e = (scale > 0.f ? scale : 1.0f / sqrtf(static_cast<float>(d_head))) * 1.4426950408889634f;
  L.q = static_cast<const __nv_bfloat16 *>(q);
  L.out = static_cast<__nv_bfloat16 *>(out);
  L.part_ml = reinterpret_cast<float *>(scratch);
  L.part_o = reinterpret_cast<float *>(scratch + ml_bytes);
  L.status = nullptr;
  L.max_parts = parts;
  switch (d_head) {
    case 64: return static_launch_d<64>(L, group, stream);
    case 128: return static_launch_d<128>(L, group, stream);
    default: return static_launch_d<256>(L, group, stream);
  }
}
