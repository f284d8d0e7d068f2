// Scaffold around the hot path (include/kvd_scaffold.h): the dense products of a decoder layer that are
// not K/V recomputation (query, output, MLP and vocabulary projections) on the recompute kernel, and the
// small elementwise steps between them.  Used by the whole-stack tests and the benchmark; nothing in
// kvd.h depends on this file.
#include <math_constants.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/kvd_scaffold.h"
#include "kvd_internal.h"
#include "kvd_ptx.cuh"

using namespace kvd;

struct kvd_linear {
  int k = 0, n = 0, n_pad = 0;
  bool norm = false;
  float rms_eps = 0.f;
  LayerState ls;  // only the prepared weight and its tensor map are used
};

static inline bool sc_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

namespace kvd {

// ---------------------------------------------------------------------------------- elementwise kernels
// One CTA per (row, query head), one thread per rotation pair.  The sum of squares over the head is
// reduced in a fixed order (shuffle tree inside a warp, warps added in index order).
__global__ void __launch_bounds__(128) kvd_query_finish_kernel(const __nv_bfloat16 *__restrict__ q_in, long long in_stride,
                                                               const int32_t *__restrict__ positions,
                                                               const __nv_bfloat16 *__restrict__ gamma_q, float eps,
                                                               const float2 *__restrict__ rope_hi,
                                                               const float2 *__restrict__ rope_lo, int max_pos,
                                                               int d_head, int n_q, int half_style,
                                                               __nv_bfloat16 *__restrict__ q_out, int *status) {
  __shared__ float s_part[4];
  const int r = blockIdx.x / n_q, h = blockIdx.x % n_q;
  const int i = threadIdx.x, half = d_head / 2;
  const int ia = half_style ? i : 2 * i, ib = half_style ? i + half : 2 * i + 1;
  const __nv_bfloat16 *src = q_in + static_cast<size_t>(r) * in_stride + static_cast<size_t>(h) * d_head;
  float a = __bfloat162float(src[ia]), b = __bfloat162float(src[ib]);
  if (gamma_q != nullptr) {
    float ss = a * a + b * b;
#pragma unroll
    for (int msk = 16; msk >= 1; msk >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, msk);
    if ((i & 31) == 0) s_part[i >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (half + 31) / 32; ++w) tot += s_part[w];
    const float rs = 1.0f / sqrtf(tot / static_cast<float>(d_head) + eps);
    a = a * rs * __bfloat162float(gamma_q[ia]);
    b = b * rs * __bfloat162float(gamma_q[ib]);
  }
  int pos = positions[r];
  if (pos < 0 || pos >= max_pos) {
    if (i == 0) atomicOr(status, STATUS_POSITION);
    pos = pos < 0 ? 0 : max_pos - 1;
  }
  // (cos, sin) of pos * f_i as the angle sum of the two table entries, as the key rotation takes it
  const float2 hi = rope_hi[static_cast<size_t>(pos >> ROPE_LO_BITS) * half + i];
  const float2 lo = rope_lo[i * ROPE_LO_SIZE + (pos & (ROPE_LO_SIZE - 1))];
  const float c = fmaf(hi.x, lo.x, -hi.y * lo.y), s = fmaf(hi.y, lo.x, hi.x * lo.y);
  __nv_bfloat16 *dst = q_out + (static_cast<size_t>(r) * n_q + h) * d_head;
  dst[ia] = __float2bfloat16_rn(fmaf(a, c, -b * s));
  dst[ib] = __float2bfloat16_rn(fmaf(a, s, b * c));
}

__global__ void __launch_bounds__(256) kvd_add_rows_kernel(uint4 *__restrict__ h, const uint4 *__restrict__ y,
                                                           long long y_stride_chunks, int m, int chunks) {
  const long long total = static_cast<long long>(m) * chunks;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = idx / chunks;
    const int c = static_cast<int>(idx % chunks);
    uint4 a = h[idx];
    const uint4 b = y[r * y_stride_chunks + c];
    uint32_t *aw = &a.x;
    const uint32_t *bw = &b.x;
#pragma unroll
    for (int j = 0; j < 4; ++j) aw[j] = pack_bf16(bf16_lo(aw[j]) + bf16_lo(bw[j]), bf16_hi(aw[j]) + bf16_hi(bw[j]));
    h[idx] = a;
  }
}

__device__ __forceinline__ float act_apply(float v, int activation) {
  if (activation == KVD_ACT_SILU) return v / (1.0f + expf(-v));
  return 0.5f * v * (1.0f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
}

__global__ void __launch_bounds__(256) kvd_gated_act_kernel(const uint4 *__restrict__ gate_up, long long stride_chunks,
                                                            int m, int width_chunks, int activation,
                                                            uint4 *__restrict__ out) {
  const long long total = static_cast<long long>(m) * width_chunks;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = idx / width_chunks;
    const int c = static_cast<int>(idx % width_chunks);
    const uint4 g = gate_up[r * stride_chunks + c];
    const uint4 u = gate_up[r * stride_chunks + width_chunks + c];
    uint4 o;
    const uint32_t *gw = &g.x, *uw = &u.x;
    uint32_t *ow = &o.x;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      ow[j] = pack_bf16(act_apply(bf16_lo(gw[j]), activation) * bf16_lo(uw[j]),
                        act_apply(bf16_hi(gw[j]), activation) * bf16_hi(uw[j]));
    out[idx] = o;
  }
}

__global__ void __launch_bounds__(256) kvd_embed_kernel(const uint4 *__restrict__ table, const int32_t *__restrict__ tokens,
                                                        int m, int chunks, int vocab, uint4 *__restrict__ out,
                                                        int *status) {
  const long long total = static_cast<long long>(m) * chunks;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = idx / chunks;
    const int c = static_cast<int>(idx % chunks);
    int t = tokens[r];
    if (t < 0 || t >= vocab) {
      if (c == 0) atomicOr(status, STATUS_POSITION);
      t = 0;
    }
    out[idx] = table[static_cast<long long>(t) * chunks + c];
  }
}

// Greedy pick in two small kernels.  (1) grid (column slices, rows): every CTA reduces its slice of a row to a
// 64-bit key -- the logit's bits mapped so that unsigned order is numeric order, above the complement of the column
// index -- and folds it into the row's slot with atomicMax: the largest value wins, among equal values the lowest
// index; the result does not depend on the order in which the CTAs arrive.  (2) one thread per row decodes the index.
constexpr int ARGMAX_SLICE = 4096;
__device__ __forceinline__ unsigned long long argmax_key(float v, int c) {
  uint32_t u = __float_as_uint(v);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // monotone map of finite floats to unsigned
  return (static_cast<unsigned long long>(u) << 32) | static_cast<uint32_t>(0x7fffffff - c);
}
__global__ void __launch_bounds__(256) kvd_argmax_slices_kernel(const __nv_bfloat16 *__restrict__ logits, long long stride, int n,
                                                                unsigned long long *__restrict__ keys) {
  __shared__ unsigned long long s_k[8];
  const __nv_bfloat16 *row = logits + static_cast<size_t>(blockIdx.y) * stride;
  const int c0 = blockIdx.x * ARGMAX_SLICE, c1 = min(n, c0 + ARGMAX_SLICE);
  unsigned long long best = 0ull;
  for (int c = c0 + threadIdx.x; c < c1; c += 256) {
    const float v = __bfloat162float(row[c]);
    if (v == v) {  // a NaN never wins
      const unsigned long long k = argmax_key(v, c);
      best = k > best ? k : best;
    }
  }
#pragma unroll
  for (int msk = 16; msk >= 1; msk >>= 1) {
    const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, msk);
    best = o > best ? o : best;
  }
  if ((threadIdx.x & 31) == 0) s_k[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) best = s_k[w] > best ? s_k[w] : best;
    if (best != 0ull) atomicMax(keys + blockIdx.y, best);
  }
}
__global__ void kvd_argmax_finish_kernel(const unsigned long long *__restrict__ keys, int m, int32_t *__restrict__ out) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < m) out[r] = keys[r] == 0ull ? 0 : 0x7fffffff - static_cast<int>(keys[r] & 0xffffffffull);
}

static unsigned grid_for(long long items, int per_block, int num_sms) {
  long long b = (items + per_block - 1) / per_block;
  const long long cap = static_cast<long long>(num_sms) * 8;
  if (b > cap) b = cap;
  return static_cast<unsigned>(b < 1 ? 1 : b);
}

}  // namespace kvd

static kvd_status sc_launched(kvd_ctx *ctx, const char *what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, what);
  ctx->launches += 1;
  return KVD_OK;
}

// ---------------------------------------------------------------------------------- dense products
extern "C" kvd_status kvd_scaffold_linear_create(kvd_ctx *ctx, const void *w, const void *gamma, int k, int n,
                                                 float rms_eps, void *stream_, kvd_linear **out) {
  if (!out) return KVD_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !w || k <= 0 || n <= 0) return KVD_ERR_INVALID_ARG;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  if (k % RC_BLOCK_K != 0) return KVD_ERR_SHAPE;
  if (gamma && !(rms_eps >= 0.f)) return KVD_ERR_INVALID_ARG;
  if (!sc_aligned16(w)) return KVD_ERR_ALIGNMENT;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  kvd_linear *lin = new (std::nothrow) kvd_linear();
  if (!lin) return KVD_ERR_CUDA;
  lin->k = k;
  lin->n = n;
  lin->n_pad = (n + ctx->block_n - 1) / ctx->block_n * ctx->block_n;
  lin->norm = gamma != nullptr;
  lin->rms_eps = rms_eps;
  const size_t bytes = static_cast<size_t>(lin->n_pad) * k * sizeof(__nv_bfloat16);
  __nv_bfloat16 *ones = nullptr;
  cudaError_t e = cudaMalloc(&lin->ls.wt, bytes);
  if (e == cudaSuccess) e = cudaMemsetAsync(lin->ls.wt, 0, bytes, stream);
  if (e == cudaSuccess && !gamma) {
    // no norm: the weight is only transposed (a scale of ones, 1.0 in bf16)
    std::vector<uint16_t> host(static_cast<size_t>(k), static_cast<uint16_t>(0x3F80));
    e = cudaMalloc(&ones, host.size() * 2);
    if (e == cudaSuccess) e = cudaMemcpy(ones, host.data(), host.size() * 2, cudaMemcpyHostToDevice);
  }
  kvd_status st = e == cudaSuccess ? KVD_OK : cuda_fail(ctx, e, "scaffold linear: allocation");
  if (st == KVD_OK)
    st = launch_prepare_weights(ctx, static_cast<const __nv_bfloat16 *>(w),
                                gamma ? static_cast<const __nv_bfloat16 *>(gamma) : ones, lin->ls.wt, k, n, stream);
  if (st == KVD_OK) st = get_rope(ctx, 10000.0f, &lin->ls.rope);  // the kernel's prologue wants a table; no row is rotated
  if (st == KVD_OK) st = encode_2d(ctx, &lin->ls.tmap_b, lin->ls.wt, k, lin->n_pad, RC_BLOCK_K, ctx->block_n / 2, 2);
  if (st == KVD_OK) {
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) st = cuda_fail(ctx, e, "scaffold linear: sync");
  }
  if (ones) cudaFree(ones);
  if (st == KVD_OK && !ctx->zero_pos) {
    e = cudaMalloc(&ctx->zero_pos, ctx->ext_sumsq_rows * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->zero_pos, 0, ctx->ext_sumsq_rows * sizeof(int32_t));
    if (e != cudaSuccess) st = cuda_fail(ctx, e, "scaffold linear: positions");
  }
  if (st != KVD_OK) {
    if (lin->ls.wt) cudaFree(lin->ls.wt);
    delete lin;
    return st;
  }
  lin->ls.set = true;
  ctx->prepared_bytes += bytes;
  *out = lin;
  return KVD_OK;
}

extern "C" void kvd_scaffold_linear_destroy(kvd_ctx *ctx, kvd_linear *lin) {
  if (!lin) return;
  if (ctx) cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  if (lin->ls.wt) cudaFree(lin->ls.wt);
  cudaGetLastError();
  delete lin;
}

extern "C" int kvd_scaffold_linear_out_cols(const kvd_linear *lin) { return lin ? lin->n_pad : 0; }

extern "C" kvd_status kvd_scaffold_linear(kvd_ctx *ctx, const kvd_linear *lin, const void *x, int m, void *out,
                                          int64_t out_row_stride, void *stream_) {
  if (!ctx || !lin || m < 0) return KVD_ERR_INVALID_ARG;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  if (m == 0) return KVD_OK;
  if (!x || !out || out_row_stride < lin->n_pad) return KVD_ERR_INVALID_ARG;
  if (!sc_aligned16(x) || !sc_aligned16(out) || out_row_stride % 8 != 0) return KVD_ERR_ALIGNMENT;
  if (static_cast<size_t>(m) > ctx->ext_sumsq_rows) return KVD_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  CUtensorMap tmap_rows;
  kvd_status st = encode_rows_3d(ctx, &tmap_rows, x, static_cast<uint64_t>(lin->k), static_cast<uint64_t>(m), 1, 2);
  if (st != KVD_OK) return st;
  static thread_local RecomputeParams p;  // large: keep it off the stack
  RcJob &J = p.jobs[0];
  J.mb_start = 0;
  J.n = m;
  J.row0 = 0;
  J.slab = -1;  // rows come from the caller's buffer
  J.positions = ctx->zero_pos;
  J.sumsq = nullptr;
  J.scale = nullptr;
  J.k_out = nullptr;  // there are no key columns
  J.v_out = static_cast<__nv_bfloat16 *>(out);
  if (!lin->norm) {
    J.sumsq = reinterpret_cast<const float *>(ctx->zero_pos);  // zeros: the row factor below comes out as exactly 1
  } else if (m > RC_INLINE_STAT_ROWS) {
    st = launch_rowstats(ctx, static_cast<const __nv_bfloat16 *>(x), ctx->ext_sumsq, m, lin->k, stream);
    if (st != KVD_OK) return st;
    J.sumsq = ctx->ext_sumsq;
  }
  p.n_jobs = 1;
  p.num_k_blocks = lin->k / RC_BLOCK_K;
  p.num_m_blocks = (m + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);
  p.num_n_blocks = lin->n_pad / ctx->block_n;
  p.k_cols = 0;  // every column is a "value" column: scaled by the row factor and stored
  p.out_row_stride = out_row_stride;
  // the row factor is 1 / sqrt(sum * inv_d_hidden + rms_eps): 1/rms(x) for a normalised product, exactly 1 otherwise
  p.inv_d_hidden = lin->norm ? 1.0f / static_cast<float>(lin->k) : 0.0f;
  p.rms_eps = lin->norm ? lin->rms_eps : 1.0f;
  p.qk_norm = 0;
  p.qk_eps = 0.f;
  p.rope_style = ctx->desc.rope_style;
  p.rope_hi = lin->ls.rope.hi;
  p.rope_lo = lin->ls.rope.lo;
  p.max_pos = 1;
  p.gamma_k = nullptr;
  p.status = ctx->d_status;
  p.timeout_ns = ctx->timeout_ns;
  p.trace = nullptr;
  p.ext_rows = static_cast<const __nv_bfloat16 *>(x);
  p.row_chunks = lin->k / 8;
  p.wide_store = (out_row_stride * 2 % 32 == 0) && ((reinterpret_cast<uintptr_t>(out) & 31u) == 0);
  p.w_scale = nullptr;
  p.rows_out_stride = out_row_stride;
  p.append_n = 0;
  p.append_rows = nullptr;
  p.append_pos = nullptr;
  p.append_sumsq = nullptr;
  p.store_rows = m;
  return launch_recompute(ctx, lin->ls, tmap_rows, tmap_rows, p, stream);
}

// ---------------------------------------------------------------------------------- elementwise steps
extern "C" kvd_status kvd_scaffold_query_finish(kvd_ctx *ctx, int layer, const void *q_in, int64_t in_row_stride,
                                                const int32_t *positions, int m, const void *gamma_q, void *q_out,
                                                void *stream_) {
  if (!ctx || m < 0 || layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (m == 0) return KVD_OK;
  const kvd_model_desc &d = ctx->desc;
  if (!q_in || !positions || !q_out || in_row_stride < static_cast<int64_t>(d.n_q_heads) * d.d_head) return KVD_ERR_INVALID_ARG;
  const int max_pos = ls.rope.n_hi * ROPE_LO_SIZE < d.max_tokens_per_seq ? ls.rope.n_hi * ROPE_LO_SIZE : d.max_tokens_per_seq;
  kvd_query_finish_kernel<<<static_cast<unsigned>(m) * d.n_q_heads, d.d_head / 2, 0, static_cast<cudaStream_t>(stream_)>>>(
      static_cast<const __nv_bfloat16 *>(q_in), in_row_stride, positions, static_cast<const __nv_bfloat16 *>(gamma_q),
      d.qk_norm_eps, ls.rope.hi, ls.rope.lo, max_pos, d.d_head, d.n_q_heads, d.rope_style == KVD_ROPE_HALF ? 1 : 0,
      static_cast<__nv_bfloat16 *>(q_out), ctx->d_status);
  return sc_launched(ctx, "launch query_finish");
}

extern "C" kvd_status kvd_scaffold_add_rows(kvd_ctx *ctx, void *h, const void *y, int64_t y_row_stride, int m, int d,
                                            void *stream_) {
  if (!ctx || m < 0 || d <= 0) return KVD_ERR_INVALID_ARG;
  if (m == 0) return KVD_OK;
  if (!h || !y || y_row_stride < d) return KVD_ERR_INVALID_ARG;
  if (d % 8 != 0 || y_row_stride % 8 != 0 || !sc_aligned16(h) || !sc_aligned16(y)) return KVD_ERR_ALIGNMENT;
  const int chunks = d / 8;
  kvd_add_rows_kernel<<<grid_for(static_cast<long long>(m) * chunks, 256, ctx->num_sms), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
      static_cast<uint4 *>(h), static_cast<const uint4 *>(y), y_row_stride / 8, m, chunks);
  return sc_launched(ctx, "launch add_rows");
}

extern "C" kvd_status kvd_scaffold_gated_act(kvd_ctx *ctx, const void *gate_up, int64_t row_stride, int m, int width,
                                             int activation, void *out, void *stream_) {
  if (!ctx || m < 0 || width <= 0) return KVD_ERR_INVALID_ARG;
  if (activation != KVD_ACT_GELU_TANH && activation != KVD_ACT_SILU) return KVD_ERR_INVALID_ARG;
  if (m == 0) return KVD_OK;
  if (!gate_up || !out || row_stride < 2 * static_cast<int64_t>(width)) return KVD_ERR_INVALID_ARG;
  if (width % 8 != 0 || row_stride % 8 != 0 || !sc_aligned16(gate_up) || !sc_aligned16(out)) return KVD_ERR_ALIGNMENT;
  const int wc = width / 8;
  kvd_gated_act_kernel<<<grid_for(static_cast<long long>(m) * wc, 256, ctx->num_sms), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
      static_cast<const uint4 *>(gate_up), row_stride / 8, m, wc, activation, static_cast<uint4 *>(out));
  return sc_launched(ctx, "launch gated_act");
}

extern "C" kvd_status kvd_scaffold_embed(kvd_ctx *ctx, const void *table, const int32_t *tokens, int m, int d, int vocab,
                                         void *out, void *stream_) {
  if (!ctx || m < 0 || d <= 0 || vocab <= 0) return KVD_ERR_INVALID_ARG;
  if (m == 0) return KVD_OK;
  if (!table || !tokens || !out) return KVD_ERR_INVALID_ARG;
  if (d % 8 != 0 || !sc_aligned16(table) || !sc_aligned16(out)) return KVD_ERR_ALIGNMENT;
  const int chunks = d / 8;
  kvd_embed_kernel<<<grid_for(static_cast<long long>(m) * chunks, 256, ctx->num_sms), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
      static_cast<const uint4 *>(table), tokens, m, chunks, vocab, static_cast<uint4 *>(out), ctx->d_status);
  return sc_launched(ctx, "launch embed");
}

extern "C" kvd_status kvd_scaffold_argmax(kvd_ctx *ctx, const void *logits, int64_t row_stride, int m, int n,
                                          int32_t *tokens_out, void *stream_) {
  if (!ctx || m < 0 || n <= 0) return KVD_ERR_INVALID_ARG;
  if (m == 0) return KVD_OK;
  if (!logits || !tokens_out || row_stride < n) return KVD_ERR_INVALID_ARG;
  if (m > 65535) return KVD_ERR_CAPACITY;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // one 64-bit slot per row, owned by the context (grown on demand; calls on a context are stream-ordered)
  if (static_cast<size_t>(m) > ctx->argmax_rows) {
    if (ctx->argmax_keys) cudaFree(ctx->argmax_keys);
    ctx->argmax_keys = nullptr;
    ctx->argmax_rows = 0;
    const size_t rows = m < 64 ? 64 : static_cast<size_t>(m);
    cudaError_t e = cudaMalloc(&ctx->argmax_keys, rows * sizeof(unsigned long long));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "scaffold argmax: scratch");
    ctx->argmax_rows = rows;
  }
  cudaError_t e = cudaMemsetAsync(ctx->argmax_keys, 0, static_cast<size_t>(m) * sizeof(unsigned long long), stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "scaffold argmax: clear");
  dim3 grid((n + ARGMAX_SLICE - 1) / ARGMAX_SLICE, m, 1);
  kvd_argmax_slices_kernel<<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16 *>(logits), row_stride, n, ctx->argmax_keys);
  kvd_status st = sc_launched(ctx, "launch argmax (slices)");
  if (st != KVD_OK) return st;
  kvd_argmax_finish_kernel<<<(m + 127) / 128, 128, 0, stream>>>(ctx->argmax_keys, m, tokens_out);
  return sc_launched(ctx, "launch argmax (finish)");
}
