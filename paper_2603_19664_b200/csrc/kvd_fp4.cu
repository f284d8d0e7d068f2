// FP4 residual checkpoints (the paper's Section 6 names lower-precision checkpoints as future work and fixes no
// format; the definition is in kvd.h): a row is stored as E2M1 codes with one E4M3 scale per block of 16 channels
// and a power-of-two scale per row, together with its position and the sum of squares of the ORIGINAL row.
// RECOMPUTE_KV from such rows expands them back to bf16 (exactly) into a caller-provided scratch and runs the
// ordinary recompute kernel on it: storage is 4-bit, the projection is the bf16 one.
#include <cuda_fp8.h>
#include <string.h>

#include "kvd_internal.h"
#include "kvd_ptx.cuh"

using namespace kvd;

namespace kvd {

constexpr int FP4_BLOCK = 16;

// E2M1 code (3 bits: exponent 2, mantissa 1; values 0, 0.5, 1, 1.5, 2, 3, 4, 6 for codes 0..7) of x / d: nearest value,
// ties to the even code, saturating at 6.  The definition rounds the fp32 quotient q = x / d and compares it with the
// midpoints 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5; here |x| is compared with midpoint * d instead, which decides the same
// way without a division per element: the products are exact (d has four significant bits, a midpoint at most three),
// and x (eight significant bits) is either equal to such a product or differs from it by far more than the rounding of
// the quotient, so fl(x / d) <= m  <=>  x <= m * d.
// (branch-free: the code is the number of midpoints passed, the comparisons alternating between > and >= so that a
// tie lands on the even code)
__device__ __forceinline__ uint32_t e2m1_code_of(float x, const float (&m)[7]) {
  const float a = fabsf(x);
  const uint32_t c = (a > m[0]) + (a >= m[1]) + (a > m[2]) + (a >= m[3]) + (a > m[4]) + (a >= m[5]) + (a > m[6]);
  return c | (x < 0.f ? 8u : 0u);
}
__device__ __forceinline__ float e2m1_value(uint32_t code) {
  const uint32_t e = (code >> 1) & 3u, m = code & 1u;
  const float mag = e == 0u ? 0.5f * static_cast<float>(m) : (1.0f + 0.5f * static_cast<float>(m)) * static_cast<float>(1u << (e - 1u));
  return (code & 8u) ? -mag : mag;
}
__device__ __forceinline__ float e4m3_value(uint32_t code) {
  return __half2float(__half(__nv_cvt_fp8_to_halfraw(static_cast<__nv_fp8_storage_t>(code), __NV_E4M3)));
}

// One warp per row.  Lane l holds chunks l, l + 32, ... (8 channels each); a block of 16 channels is a pair of
// neighbouring chunks, i.e. an even lane and its odd neighbour.  Rows of up to 32 * CPL chunks stay in registers.
template <int CPL>
__global__ void __launch_bounds__(256, 2) kvd_checkpoint_fp4_kernel(const uint4 *__restrict__ rows, const int32_t *__restrict__ pos,
                                                                 uint32_t *__restrict__ dst_codes, uint8_t *__restrict__ dst_block,
                                                                 int32_t *__restrict__ dst_pos, float *__restrict__ dst_sumsq,
                                                                 float *__restrict__ dst_scale, int row_chunks, int n) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    const size_t off = static_cast<size_t>(r) * row_chunks;
    uint4 v[CPL];
    float cmax[CPL], amax = 0.f;
    uint64_t ps2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = lane + 32 * i;
      v[i] = c < row_chunks ? __ldg(rows + off + c) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      sumsq_chunk(ps2, v[i]);  // the lane's chunks in ascending order, as every other taker of the statistic does
      const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
      float m = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) m = fmaxf(m, fmaxf(fabsf(bf16_lo(w[j])), fabsf(bf16_hi(w[j]))));
      cmax[i] = m;
      amax = fmaxf(amax, m);
    }
    const float ss = sumsq_finish(ps2);
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, k));
    // row scale 2^(floor(log2(amax)) - 10); 1 for an all-zero row
    int ex = 0;
    frexpf(amax, &ex);  // amax = m * 2^ex, m in [0.5, 1)
    const float s_row = amax > 0.f ? ldexpf(1.0f, ex - 1 - 10) : 1.0f;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = lane + 32 * i;
      const float bmax = fmaxf(cmax[i], __shfl_xor_sync(0xffffffffu, cmax[i], 1));
      const float t = __fdiv_rn(__fdiv_rn(bmax, 6.0f), s_row);
      const uint32_t bcode = __nv_cvt_float2_to_fp8x2(make_float2(t, 0.f), __NV_SATFINITE, __NV_E4M3) & 0xffu;
      const float d = __fmul_rn(e4m3_value(bcode), s_row);
      const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
      const float mid[7] = {0.25f * d, 0.75f * d, 1.25f * d, 1.75f * d, 2.5f * d, 3.5f * d, 5.0f * d};  // exact products
      uint32_t packed = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        packed |= (e2m1_code_of(bf16_lo(w[j]), mid) | (e2m1_code_of(bf16_hi(w[j]), mid) << 4)) << (8 * j);  // channel 2j in the low nibble of byte j
      if (!(d > 0.f)) packed = 0;  // a block whose scale rounded to zero has all codes zero
      if (c < row_chunks) {
        dst_codes[off + c] = packed;
        if ((lane & 1) == 0) dst_block[static_cast<size_t>(r) * (row_chunks / 2) + (c >> 1)] = static_cast<uint8_t>(bcode);
      }
    }
    if (lane == 0) {
      dst_scale[r] = s_row;
      dst_sumsq[r] = ss;
      dst_pos[r] = pos[r];
    }
  }
}

// Expand ranges of the FP4 store into bf16 rows (exact), with their positions and statistics, for the ordinary
// recompute kernel.  Row i of the launch belongs to the last range whose first scratch row is <= i.
struct Fp4Ranges {
  int n_ranges;
  int total_rows;
  int dst0[KVD_MAX_STORE_RANGES + 1];      // first scratch row of each range (ascending), then the total
  long long slot0[KVD_MAX_STORE_RANGES];   // first store slot of each range
};
__global__ void __launch_bounds__(256) kvd_expand_fp4_kernel(const uint32_t *__restrict__ codes, const uint8_t *__restrict__ block,
                                                             const int32_t *__restrict__ spos, const float *__restrict__ ssumsq,
                                                             const float *__restrict__ sscale, uint4 *__restrict__ out_rows,
                                                             int32_t *__restrict__ out_pos, float *__restrict__ out_sumsq,
                                                             int row_chunks, const __grid_constant__ Fp4Ranges R) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  grid_launch_dependents();
  for (int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < R.total_rows; i += warps) {
    int lo = 0, hi = R.n_ranges;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (R.dst0[mid] <= i) lo = mid;
      else hi = mid;
    }
    const size_t slot = static_cast<size_t>(R.slot0[lo]) + (i - R.dst0[lo]);
    const float s_row = __ldg(sscale + slot);
    for (int c = lane; c < row_chunks; c += 32) {
      const uint32_t packed = __ldg(codes + slot * row_chunks + c);
      const float d = __fmul_rn(e4m3_value(__ldg(block + slot * (row_chunks / 2) + (c >> 1))), s_row);
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t b = (packed >> (8 * j)) & 0xffu;
        w[j] = pack_bf16(e2m1_value(b & 0xfu) * d, e2m1_value(b >> 4) * d);  // exact products, exact in bf16
      }
      out_rows[static_cast<size_t>(i) * row_chunks + c] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (lane == 0) {
      out_pos[i] = __ldg(spos + slot);
      out_sumsq[i] = __ldg(ssumsq + slot);
    }
  }
}

static inline size_t ru256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace kvd

static bool fp4_shape_ok(const kvd_model_desc *d) { return d->d_hidden % 64 == 0; }  // whole blocks, 16-byte code rows

extern "C" size_t kvd_store_bytes_fp4(const kvd_model_desc *d, int layers_stored) {
  if (!d || layers_stored <= 0 || kvd_store_bytes(d, 1) == 0 || !fp4_shape_ok(d)) return 0;
  const size_t slots = static_cast<size_t>(layers_stored) * d->max_seqs * d->max_tokens_per_seq;
  // codes, block scales, then positions, sums of squares and row scales, each region at a 256-byte multiple
  return ru256(slots * d->d_hidden / 2) + ru256(slots * d->d_hidden / FP4_BLOCK) + 3 * ru256(slots * 4);
}

extern "C" size_t kvd_fp4_scratch_bytes(const kvd_model_desc *d, int max_rows) {
  if (!d || max_rows <= 0 || kvd_store_bytes(d, 1) == 0 || !fp4_shape_ok(d)) return 0;
  return ru256(static_cast<size_t>(max_rows) * d->d_hidden * 2) + 2 * ru256(static_cast<size_t>(max_rows) * 4);
}

extern "C" kvd_status kvd_attach_store_fp4(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored) {
  if (!ctx || !arena || layers_stored <= 0 || layers_stored > ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return KVD_ERR_ALIGNMENT;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  const size_t need = kvd_store_bytes_fp4(&ctx->desc, layers_stored);
  if (need == 0) return KVD_ERR_SHAPE;
  if (bytes < need) return KVD_ERR_CAPACITY;
  const kvd_model_desc &d = ctx->desc;
  const size_t slots = static_cast<size_t>(layers_stored) * d.max_seqs * d.max_tokens_per_seq;
  uint8_t *base = static_cast<uint8_t *>(arena);
  ctx->store4_codes = base;
  ctx->store4_block = base + ru256(slots * d.d_hidden / 2);
  ctx->store4_pos = reinterpret_cast<int32_t *>(ctx->store4_block + ru256(slots * d.d_hidden / FP4_BLOCK));
  ctx->store4_sumsq = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(ctx->store4_pos) + ru256(slots * 4));
  ctx->store4_scale = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(ctx->store4_sumsq) + ru256(slots * 4));
  ctx->layers_stored4 = layers_stored;
  ctx->rows_stored4.assign(static_cast<size_t>(layers_stored) * d.max_seqs, 0);
  return KVD_OK;
}

extern "C" int kvd_rows_stored_fp4(const kvd_ctx *ctx, int layer, int seq) {
  if (!ctx || !ctx->store4_codes || layer < 0 || layer >= ctx->layers_stored4 || seq < 0 || seq >= ctx->desc.max_seqs) return -1;
  return ctx->rows_stored4[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
}

extern "C" kvd_status kvd_reset_sequence_fp4(kvd_ctx *ctx, int seq) {
  if (!ctx || seq < 0 || seq >= ctx->desc.max_seqs) return KVD_ERR_INVALID_ARG;
  if (!ctx->store4_codes) return KVD_ERR_STATE;
  for (int l = 0; l < ctx->layers_stored4; ++l) ctx->rows_stored4[static_cast<size_t>(l) * ctx->desc.max_seqs + seq] = 0;
  return KVD_OK;
}

static inline size_t fp4_slot(const kvd_ctx *ctx, int layer, int seq) {
  return (static_cast<size_t>(layer) * ctx->desc.max_seqs + seq) * ctx->desc.max_tokens_per_seq;
}

extern "C" kvd_status kvd_checkpoint_residual_fp4(kvd_ctx *ctx, int seq, int layer, const void *rows, const int32_t *positions,
                                                  int n, void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (!ctx->store4_codes) return KVD_ERR_STATE;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;  // the quantiser reads bf16 rows
  if (seq < 0 || seq >= ctx->desc.max_seqs || layer < 0 || layer >= ctx->layers_stored4) return KVD_ERR_INVALID_ARG;
  if (n == 0) return KVD_OK;
  if (!rows || !positions) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(rows) & 15u) != 0) return KVD_ERR_ALIGNMENT;
  int &count = ctx->rows_stored4[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
  if (count + n > ctx->desc.max_tokens_per_seq) return KVD_ERR_CAPACITY;
  const size_t slot = fp4_slot(ctx, layer, seq) + count;
  const int d = ctx->desc.d_hidden, row_chunks = d / 8;
  long long blocks = (static_cast<long long>(n) + 7) / 8;
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint32_t *dc = reinterpret_cast<uint32_t *>(ctx->store4_codes + slot * (d / 2));
  uint8_t *db = ctx->store4_block + slot * (d / FP4_BLOCK);
  const uint4 *src = static_cast<const uint4 *>(rows);
  if (row_chunks <= 320)
    kvd_checkpoint_fp4_kernel<10><<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        src, positions, dc, db, ctx->store4_pos + slot, ctx->store4_sumsq + slot, ctx->store4_scale + slot, row_chunks, n);
  else
    return KVD_ERR_SHAPE;  // rows wider than 2560 channels are not held in registers
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch checkpoint_fp4");
  ctx->launches += 1;
  count += n;
  return KVD_OK;
}

extern "C" kvd_status kvd_recompute_kv_fp4(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                           int64_t out_row_stride, void *scratch, size_t scratch_bytes, void *stream_) {
  if (!ctx || n_ranges < 0 || n_ranges > KVD_MAX_STORE_RANGES || (n_ranges > 0 && !ranges)) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  if (out_row_stride < kdim) return KVD_ERR_INVALID_ARG;
  if (out_row_stride % 8 != 0) return KVD_ERR_ALIGNMENT;
  static thread_local RecomputeParams p;  // large: keep it off the stack
  Fp4Ranges R;
  int n_jobs = 0, mb = 0, total = 0;
  for (int i = 0; i < n_ranges; ++i) {
    const kvd_store_range &r = ranges[i];
    if (r.n < 0) return KVD_ERR_INVALID_ARG;
    if (r.n == 0) continue;
    if (!ctx->store4_codes) return KVD_ERR_STATE;
    if (r.seq < 0 || r.seq >= d.max_seqs || layer >= ctx->layers_stored4 || r.first_row < 0) return KVD_ERR_INVALID_ARG;
    if (!r.k_out || !r.v_out) return KVD_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(r.k_out) | reinterpret_cast<uintptr_t>(r.v_out)) & 15u) != 0) return KVD_ERR_ALIGNMENT;
    const int have = ctx->rows_stored4[static_cast<size_t>(layer) * d.max_seqs + r.seq];
    if (r.first_row > have || r.n > have - r.first_row) return KVD_ERR_CAPACITY;
    R.dst0[n_jobs] = total;
    R.slot0[n_jobs] = static_cast<long long>(fp4_slot(ctx, layer, r.seq) + r.first_row);
    RcJob &J = p.jobs[n_jobs++];
    J.mb_start = mb;
    J.n = r.n;
    J.row0 = total;  // first row of this range in the scratch
    J.slab = -1;     // the expanded rows are "caller rows" to the recompute kernel
    J.scale = nullptr;
    J.k_out = static_cast<__nv_bfloat16 *>(r.k_out);
    J.v_out = static_cast<__nv_bfloat16 *>(r.v_out);
    mb += (r.n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);
    total += r.n;
  }
  if (n_jobs == 0) return KVD_OK;
  if (!scratch) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return KVD_ERR_ALIGNMENT;
  if (scratch_bytes < kvd_fp4_scratch_bytes(&d, total)) return KVD_ERR_CAPACITY;
  R.n_ranges = n_jobs;
  R.total_rows = total;
  R.dst0[n_jobs] = total;
  uint8_t *sb = static_cast<uint8_t *>(scratch);
  __nv_bfloat16 *x = reinterpret_cast<__nv_bfloat16 *>(sb);
  // the regions are laid out for `total` rows: rows, then sums of squares, then positions
  float *xs = reinterpret_cast<float *>(sb + ru256(static_cast<size_t>(total) * d.d_hidden * 2));
  int32_t *xp = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(xs) + ru256(static_cast<size_t>(total) * 4));
  for (int j = 0; j < n_jobs; ++j) {
    p.jobs[j].positions = xp + p.jobs[j].row0;
    p.jobs[j].sumsq = xs + p.jobs[j].row0;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int row_chunks = d.d_hidden / 8;
  long long blocks = (static_cast<long long>(total) + 7) / 8;
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  kvd_expand_fp4_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
      reinterpret_cast<const uint32_t *>(ctx->store4_codes), ctx->store4_block, ctx->store4_pos, ctx->store4_sumsq,
      ctx->store4_scale, reinterpret_cast<uint4 *>(x), xp, xs, row_chunks, R);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "launch expand_fp4");
  ctx->launches += 1;
  CUtensorMap tmap_rows;
  kvd_status st = encode_rows_3d(ctx, &tmap_rows, x, d.d_hidden, static_cast<uint64_t>(total), 1, 2);
  if (st != KVD_OK) return st;
  p.n_jobs = n_jobs;
  p.num_k_blocks = d.d_hidden / RC_BLOCK_K;
  p.num_m_blocks = mb;
  p.num_n_blocks = 2 * kdim / ctx->block_n;
  p.k_cols = kdim;
  p.out_row_stride = out_row_stride;
  p.rows_out_stride = out_row_stride;
  p.inv_d_hidden = 1.0f / static_cast<float>(d.d_hidden);
  p.rms_eps = d.rms_eps;
  p.qk_norm = d.qk_norm;
  p.qk_eps = d.qk_norm_eps;
  p.rope_style = d.rope_style;
  p.rope_hi = ls.rope.hi;
  p.rope_lo = ls.rope.lo;
  p.max_pos = ls.rope.n_hi * ROPE_LO_SIZE < d.max_tokens_per_seq ? ls.rope.n_hi * ROPE_LO_SIZE : d.max_tokens_per_seq;
  p.gamma_k = d.qk_norm ? ls.gamma_k : nullptr;
  p.status = ctx->d_status;
  p.timeout_ns = ctx->timeout_ns;
  p.trace = nullptr;
  p.ext_rows = x;
  p.row_chunks = row_chunks;
  p.w_scale = nullptr;
  p.store_rows = total;
  p.append_n = 0;
  p.append_rows = nullptr;
  p.append_pos = nullptr;
  p.append_sumsq = nullptr;
  p.wide_store = out_row_stride * 2 % 32 == 0;
  for (int j = 0; j < n_jobs; ++j)
    if (((reinterpret_cast<uintptr_t>(p.jobs[j].k_out) | reinterpret_cast<uintptr_t>(p.jobs[j].v_out)) & 31u) != 0) p.wide_store = 0;
  return launch_recompute(ctx, ls, tmap_rows, tmap_rows, p, stream);
}
