// C ABI of the KV-Direct hot path: context management, argument validation, launch set-up.
// All arithmetic of the method lives in the kernels; nothing here computes K, V or attention.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "kvd_internal.h"

using namespace kvd;

namespace kvd {
kvd_status cuda_fail(kvd_ctx *ctx, cudaError_t e, const char *where) {
  if (ctx) {
    ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
  }
  return KVD_ERR_CUDA;
}
}  // namespace kvd

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static kvd_status check_desc(const kvd_model_desc *d) {
  if (!d) return KVD_ERR_INVALID_ARG;
  if (d->n_layers <= 0 || d->d_hidden <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->max_seqs <= 0 ||
      d->max_tokens_per_seq <= 0 || d->max_batch <= 0)
    return KVD_ERR_INVALID_ARG;
  if (!(d->rms_eps >= 0.f) || !(d->qk_norm_eps >= 0.f)) return KVD_ERR_INVALID_ARG;
  if (d->rope_style != KVD_ROPE_INTERLEAVED && d->rope_style != KVD_ROPE_HALF) return KVD_ERR_INVALID_ARG;
  if (d->d_hidden % 64 != 0) return KVD_ERR_SHAPE;
  if (d->d_head != 64 && d->d_head != 128 && d->d_head != 256) return KVD_ERR_SHAPE;
  if (d->n_q_heads % d->n_kv_heads != 0) return KVD_ERR_SHAPE;
  const int g = d->n_q_heads / d->n_kv_heads;
  if (!(g == 1 || g == 2 || g == 3 || g == 4 || g == 8)) return KVD_ERR_SHAPE;
  if ((2 * d->n_kv_heads * d->d_head) % 128 != 0) return KVD_ERR_SHAPE;
  return KVD_OK;
}

static int pick_block_n(const kvd_model_desc *d) {
  const int n = 2 * d->n_kv_heads * d->d_head;
  if (n % 256 == 0) return 256;
  return 128;  // n % 128 == 0 was checked; d_head <= 128 follows because 2*n_kv*256 is a multiple of 256
}

extern "C" const char *kvd_version(void) { return "0.1"; }

extern "C" const char *kvd_status_string(kvd_status s) {
  switch (s) {
    case KVD_OK: return "ok";
    case KVD_ERR_INVALID_ARG: return "invalid argument";
    case KVD_ERR_SHAPE: return "unsupported shape";
    case KVD_ERR_ALIGNMENT: return "misaligned pointer or stride";
    case KVD_ERR_CAPACITY: return "capacity exceeded";
    case KVD_ERR_STATE: return "call made in the wrong state";
    case KVD_ERR_UNSUPPORTED: return "no usable sm_100 device";
    case KVD_ERR_CUDA: return "CUDA error";
    case KVD_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case KVD_ERR_POSITION: return "row position out of range";
    case KVD_ERR_BOUNDS: return "an index test of the checking build failed";
  }
  return "unknown status";
}

static inline int dtype_bytes(int dtype) { return dtype == KVD_DTYPE_F32 ? 4 : 2; }

extern "C" size_t kvd_store_bytes_dtype(const kvd_model_desc *d, int layers_stored, int dtype) {
  if (check_desc(d) != KVD_OK || layers_stored <= 0) return 0;
  if (dtype != KVD_DTYPE_BF16 && dtype != KVD_DTYPE_F16 && dtype != KVD_DTYPE_F32) return 0;
  const size_t slots = static_cast<size_t>(layers_stored) * d->max_seqs * d->max_tokens_per_seq;
  // rows, then positions, then the rows' sums of squares, each region starting at a 256-byte multiple
  return round_up(slots * d->d_hidden * dtype_bytes(dtype), 256) + 2 * round_up(slots * 4, 256);
}

extern "C" size_t kvd_store_bytes(const kvd_model_desc *d, int layers_stored) {
  return kvd_store_bytes_dtype(d, layers_stored, KVD_DTYPE_BF16);
}

// chunk partials of one sequence
static size_t parts_per_seq(const kvd_model_desc *d) {
  // the streaming kernel's chunks plus, for kvd_decode_attention_recompute, one partial per 256-row block
  // of a recomputed range
  return attn_max_chunks(d->d_head, d->n_kv_heads, d->max_tokens_per_seq) + (d->max_tokens_per_seq + 255) / 256;
}

extern "C" size_t kvd_workspace_bytes(const kvd_model_desc *d) {
  if (check_desc(d) != KVD_OK) return 0;
  const size_t parts = static_cast<size_t>(d->max_batch) * parts_per_seq(d);
  return round_up(parts * d->n_q_heads * d->d_head * 4, 256) + round_up(parts * d->n_q_heads * 2 * 4, 256);
}

extern "C" int kvd_attention_split(int d_head, int n_kv_heads, int first_visible, int last_visible, int *chunk_keys) {
  if ((d_head != 64 && d_head != 128 && d_head != 256) || n_kv_heads < 1) return 0;
  if (first_visible < 0 || last_visible < first_visible) return 0;
  const int iters = attn_iters_for_span(d_head, n_kv_heads, last_visible - first_visible + 1);
  const int ck = attn_chunk_keys(d_head, iters);
  if (chunk_keys) *chunk_keys = ck;
  return last_visible / ck - first_visible / ck + 1;
}

extern "C" kvd_status kvd_create(const kvd_model_desc *desc, kvd_ctx **out) {
  if (!out) return KVD_ERR_INVALID_ARG;
  *out = nullptr;
  kvd_status st = check_desc(desc);
  if (st != KVD_OK) return st;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return KVD_ERR_UNSUPPORTED;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    cudaGetLastError();
    return KVD_ERR_UNSUPPORTED;
  }
  if (prop.major != 10) return KVD_ERR_UNSUPPORTED;
  kvd_ctx *ctx = new (std::nothrow) kvd_ctx();
  if (!ctx) return KVD_ERR_CUDA;
  ctx->desc = *desc;
  ctx->device = dev;
  ctx->num_sms = prop.multiProcessorCount;
  ctx->block_n = pick_block_n(desc);
  ctx->layers.resize(desc->n_layers);
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    delete ctx;
    return KVD_ERR_UNSUPPORTED;
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  cudaError_t e = cudaMalloc(&ctx->d_status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int));
  if (e == cudaSuccess) {
    // scratch for the statistics of caller rows (one fp32 per row, at most one full batch of rows)
    ctx->ext_sumsq_rows = static_cast<size_t>(desc->max_seqs) * desc->max_tokens_per_seq;
    e = cudaMalloc(&ctx->ext_sumsq, ctx->ext_sumsq_rows * sizeof(float));
    if (e == cudaSuccess) ctx->prepared_bytes += ctx->ext_sumsq_rows * sizeof(float);
  }
  if (e != cudaSuccess) {
    cudaFree(ctx->d_status);
    delete ctx;
    return KVD_ERR_CUDA;
  }
  const char *env = getenv("KVD_SPIN_LIMIT_MS");
  if (env) {
    const long ms = atol(env);
    if (ms > 0) ctx->timeout_ns = static_cast<unsigned long long>(ms) * 1000000ull;
  }
  *out = ctx;
  return KVD_OK;
}

extern "C" void kvd_destroy(kvd_ctx *ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  for (auto &l : ctx->layers) {
    if (l.wt) cudaFree(l.wt);
    if (l.gamma_k) cudaFree(l.gamma_k);
    if (l.wt8) cudaFree(l.wt8);
    if (l.w_scale8) cudaFree(l.w_scale8);
  }
  for (auto &kv : ctx->rope_cache) {
    if (kv.second.hi) cudaFree(kv.second.hi);
    if (kv.second.lo) cudaFree(kv.second.lo);
  }
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->ext_sumsq) cudaFree(ctx->ext_sumsq);
  if (ctx->zero_pos) cudaFree(ctx->zero_pos);
  if (ctx->argmax_keys) cudaFree(ctx->argmax_keys);
  if (ctx->amax_scratch) cudaFree(ctx->amax_scratch);
  cudaGetLastError();
  delete ctx;
}

// (eb = bytes per element: 2 for bf16, 1 for the FP8 variant's codes; a box row is 128 bytes either way)
namespace kvd {
// element type of a tensor map for `eb` bytes per element (16-bit maps follow the context's type; the copies
// are bit-for-bit either way)
static CUtensorMapDataType map_type(const kvd_ctx *ctx, int eb) {
  if (eb == 4) return CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  if (eb == 1) return CU_TENSOR_MAP_DATA_TYPE_UINT8;
  return ctx->dtype == KVD_DTYPE_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
}

kvd_status encode_2d(kvd_ctx *ctx, CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer,
                     uint32_t box_inner, uint32_t box_outer, int eb) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * eb};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(map, map_type(ctx, eb), 2,
                           const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char buf[64];
    snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed: %d", static_cast<int>(r));
    ctx->last_error = buf;
    return KVD_ERR_CUDA;
  }
  return KVD_OK;
}

// Row source of the recompute GEMM as a 3-D map [slabs][rows][d_hidden]; box = one 128 x 64 tile.
kvd_status encode_rows_3d(kvd_ctx *ctx, CUtensorMap *map, const void *base, uint64_t d_hidden, uint64_t rows,
                          uint64_t slabs, int eb) {
  cuuint64_t dims[3] = {d_hidden, rows, slabs};
  cuuint64_t strides[2] = {d_hidden * eb, rows * d_hidden * eb};
  cuuint32_t box[3] = {static_cast<cuuint32_t>(RC_BLOCK_K * 2 / eb), RC_BLOCK_M, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ctx->encode(map, map_type(ctx, eb), 3,
                           const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char buf[64];
    snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled (rows) failed: %d", static_cast<int>(r));
    ctx->last_error = buf;
    return KVD_ERR_CUDA;
  }
  return KVD_OK;
}

// (cos, sin) tables of Eq. 11-12 split as position = 16*hi + lo; built in double on the host.
// hi is row-major [hi][pair]; lo is pair-major [pair][lo] so that neighbouring positions read
// neighbouring shared-memory words.
kvd_status get_rope(kvd_ctx *ctx, float theta, RopeTable *out) {
  uint32_t key;
  memcpy(&key, &theta, 4);
  auto it = ctx->rope_cache.find(key);
  if (it != ctx->rope_cache.end()) {
    *out = it->second;
    return KVD_OK;
  }
  const int half = ctx->desc.d_head / 2;
  const int n_hi = (ctx->desc.max_tokens_per_seq + ROPE_LO_SIZE - 1) / ROPE_LO_SIZE;
  std::vector<float2> hi(static_cast<size_t>(n_hi) * half), lo(static_cast<size_t>(ROPE_LO_SIZE) * half);
  for (int i = 0; i < half; ++i) {
    const double freq = pow(static_cast<double>(theta), -2.0 * i / ctx->desc.d_head);
    for (int h = 0; h < n_hi; ++h) {
      const double a = static_cast<double>(h) * ROPE_LO_SIZE * freq;
      hi[static_cast<size_t>(h) * half + i] = make_float2(static_cast<float>(cos(a)), static_cast<float>(sin(a)));
    }
    for (int l = 0; l < ROPE_LO_SIZE; ++l) {
      const double a = static_cast<double>(l) * freq;
      lo[static_cast<size_t>(i) * ROPE_LO_SIZE + l] = make_float2(static_cast<float>(cos(a)), static_cast<float>(sin(a)));
    }
  }
  RopeTable t;
  t.n_hi = n_hi;
  cudaError_t e = cudaMalloc(&t.hi, hi.size() * sizeof(float2));
  if (e == cudaSuccess) e = cudaMalloc(&t.lo, lo.size() * sizeof(float2));
  if (e == cudaSuccess) e = cudaMemcpy(t.hi, hi.data(), hi.size() * sizeof(float2), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(t.lo, lo.data(), lo.size() * sizeof(float2), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "rope tables");
  ctx->prepared_bytes += (hi.size() + lo.size()) * sizeof(float2);
  ctx->rope_cache[key] = t;
  *out = t;
  return KVD_OK;
}
}  // namespace kvd

extern "C" kvd_status kvd_set_dtype(kvd_ctx *ctx, int dtype) {
  if (!ctx || (dtype != KVD_DTYPE_BF16 && dtype != KVD_DTYPE_F16 && dtype != KVD_DTYPE_F32)) return KVD_ERR_INVALID_ARG;
  for (const LayerState &l : ctx->layers)
    if (l.set) return KVD_ERR_STATE;  // weights are prepared in the element type: choose it first
  if (ctx->store_rows && dtype_bytes(dtype) != dtype_bytes(ctx->dtype)) return KVD_ERR_STATE;  // the store is laid out for it
  for (int c : ctx->rows_stored)
    if (c != 0) return KVD_ERR_STATE;
  // the FP8 variant reads bf16 rows and bf16-folded weights: no other element type next to an FP8 store
  if (dtype != KVD_DTYPE_BF16 && (ctx->store8_codes || ctx->store4_codes)) return KVD_ERR_STATE;
  for (int c : ctx->rows_stored8)
    if (c != 0) return KVD_ERR_STATE;
  ctx->dtype = dtype;
  return KVD_OK;
}

extern "C" kvd_status kvd_set_layer(kvd_ctx *ctx, int layer, const kvd_layer_desc *ld, void *stream_) {
  if (!ctx || !ld) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if (!ld->w_kv || !ld->gamma_in) return KVD_ERR_INVALID_ARG;
  if (ctx->desc.qk_norm && !ld->gamma_k) return KVD_ERR_INVALID_ARG;
  if (!(ld->rope_theta > 1.0f) || ld->sliding_window < 0) return KVD_ERR_INVALID_ARG;
  if (!aligned16(ld->w_kv)) return KVD_ERR_ALIGNMENT;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const kvd_model_desc &d = ctx->desc;
  const int n_cols = 2 * d.n_kv_heads * d.d_head;
  LayerState &ls = ctx->layers[layer];
  cudaError_t e;
  if (!ls.wt) {
    e = cudaMalloc(&ls.wt, static_cast<size_t>(n_cols) * d.d_hidden * dtype_bytes(ctx->dtype));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc(prepared weights)");
    ctx->prepared_bytes += static_cast<size_t>(n_cols) * d.d_hidden * dtype_bytes(ctx->dtype);
  }
  if (d.qk_norm && !ls.gamma_k) {
    e = cudaMalloc(&ls.gamma_k, d.d_head * sizeof(float));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc(gamma_k)");
    ctx->prepared_bytes += d.d_head * sizeof(float);
  }
  kvd_status st = launch_prepare_weights(ctx, static_cast<const __nv_bfloat16 *>(ld->w_kv),
                                         static_cast<const __nv_bfloat16 *>(ld->gamma_in), ls.wt, d.d_hidden, n_cols,
                                         stream);
  if (st != KVD_OK) return st;
  if (d.qk_norm) {
    st = launch_convert_gamma(ctx, static_cast<const __nv_bfloat16 *>(ld->gamma_k), ls.gamma_k, d.d_head, stream);
    if (st != KVD_OK) return st;
  }
  st = get_rope(ctx, ld->rope_theta, &ls.rope);
  if (st != KVD_OK) return st;
  // half tile per CTA, 128 bytes of channels per k block
  st = encode_2d(ctx, &ls.tmap_b, ls.wt, d.d_hidden, n_cols, RC_BLOCK_K * 2 / dtype_bytes(ctx->dtype), ctx->block_n / 2,
                 dtype_bytes(ctx->dtype));
  if (st != KVD_OK) return st;
  // the FP8 variant's copy of W' (E4M3 codes and one scale); rows of d_hidden bytes must be TMA-addressable
  if (d.d_hidden % 16 == 0 && ctx->dtype == KVD_DTYPE_BF16) {
    if (!ls.wt8) {
      e = cudaMalloc(&ls.wt8, static_cast<size_t>(n_cols) * d.d_hidden);
      if (e == cudaSuccess) e = cudaMalloc(&ls.w_scale8, sizeof(float));
      if (e == cudaSuccess && !ctx->amax_scratch) e = cudaMalloc(&ctx->amax_scratch, sizeof(unsigned));
      if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc(fp8 weights)");
      ctx->prepared_bytes += static_cast<size_t>(n_cols) * d.d_hidden + sizeof(float);
    }
    st = launch_prepare_weights_fp8(ctx, static_cast<const __nv_bfloat16 *>(ld->w_kv),
                                    static_cast<const __nv_bfloat16 *>(ld->gamma_in), ls.wt8, d.d_hidden, n_cols,
                                    ctx->amax_scratch, ls.w_scale8, stream);
    if (st != KVD_OK) return st;
    st = encode_2d(ctx, &ls.tmap_b8, ls.wt8, d.d_hidden, n_cols, 2 * RC_BLOCK_K, ctx->block_n / 2, 1);
    if (st != KVD_OK) return st;
  }
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "kvd_set_layer sync");
  ls.theta = ld->rope_theta;
  ls.window = ld->sliding_window;
  ls.set = true;
  return KVD_OK;
}

extern "C" kvd_status kvd_attach_store(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored) {
  if (!ctx || !arena || layers_stored <= 0 || layers_stored > ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return KVD_ERR_ALIGNMENT;
  const size_t need = kvd_store_bytes_dtype(&ctx->desc, layers_stored, ctx->dtype);
  if (bytes < need) return KVD_ERR_CAPACITY;
  const kvd_model_desc &d = ctx->desc;
  const int es = dtype_bytes(ctx->dtype), ew = es / 2;  // store_rows counts 16-bit units
  const size_t slots = static_cast<size_t>(layers_stored) * d.max_seqs * d.max_tokens_per_seq;
  ctx->store_rows = static_cast<__nv_bfloat16 *>(arena);
  ctx->store_pos = reinterpret_cast<int32_t *>(static_cast<uint8_t *>(arena) + round_up(slots * d.d_hidden * es, 256));
  ctx->store_sumsq = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(ctx->store_pos) + round_up(slots * 4, 256));
  ctx->layers_stored = layers_stored;
  ctx->rows_stored.assign(static_cast<size_t>(layers_stored) * d.max_seqs, 0);
  ctx->store_maps.resize(layers_stored);
  for (int l = 0; l < layers_stored; ++l) {
    const __nv_bfloat16 *base = ctx->store_rows + static_cast<size_t>(l) * d.max_seqs * d.max_tokens_per_seq * d.d_hidden * ew;
    kvd_status st = encode_rows_3d(ctx, &ctx->store_maps[l], base, d.d_hidden, d.max_tokens_per_seq, d.max_seqs, es);
    if (st != KVD_OK) {
      ctx->store_rows = nullptr;
      ctx->layers_stored = 0;
      return st;
    }
  }
  return KVD_OK;
}

extern "C" kvd_status kvd_reset_sequence(kvd_ctx *ctx, int seq) {
  if (!ctx || seq < 0 || seq >= ctx->desc.max_seqs) return KVD_ERR_INVALID_ARG;
  if (!ctx->store_rows) return KVD_ERR_STATE;
  for (int l = 0; l < ctx->layers_stored; ++l) ctx->rows_stored[static_cast<size_t>(l) * ctx->desc.max_seqs + seq] = 0;
  return KVD_OK;
}

extern "C" kvd_status kvd_reset_sequence_fp8(kvd_ctx *ctx, int seq) {
  if (!ctx || seq < 0 || seq >= ctx->desc.max_seqs) return KVD_ERR_INVALID_ARG;
  if (!ctx->store8_codes) return KVD_ERR_STATE;
  for (int l = 0; l < ctx->layers_stored8; ++l) ctx->rows_stored8[static_cast<size_t>(l) * ctx->desc.max_seqs + seq] = 0;
  return KVD_OK;
}

extern "C" int kvd_rows_stored(const kvd_ctx *ctx, int layer, int seq) {
  if (!ctx || !ctx->store_rows || layer < 0 || layer >= ctx->layers_stored || seq < 0 || seq >= ctx->desc.max_seqs)
    return -1;
  return ctx->rows_stored[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
}

extern "C" kvd_status kvd_attach_workspace(kvd_ctx *ctx, void *ws, size_t bytes) {
  if (!ctx || !ws) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return KVD_ERR_ALIGNMENT;
  const size_t need = kvd_workspace_bytes(&ctx->desc);
  if (bytes < need) return KVD_ERR_CAPACITY;
  const kvd_model_desc &d = ctx->desc;
  const size_t parts = static_cast<size_t>(d.max_batch) * parts_per_seq(&d);
  ctx->part_o = static_cast<float *>(ws);
  uint8_t *base = static_cast<uint8_t *>(ws);
  ctx->part_ml = reinterpret_cast<float *>(base + round_up(parts * d.n_q_heads * d.d_head * 4, 256));
  ctx->max_parts = static_cast<int>(parts);
  ctx->workspace_bytes = need;
  return KVD_OK;
}

static inline size_t store_slot(const kvd_ctx *ctx, int layer, int seq) {
  return (static_cast<size_t>(layer) * ctx->desc.max_seqs + seq) * ctx->desc.max_tokens_per_seq;
}

extern "C" kvd_status kvd_checkpoint_residual(kvd_ctx *ctx, int seq, int layer, const void *rows,
                                              const int32_t *positions, int n, void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (!ctx->store_rows) return KVD_ERR_STATE;
  if (seq < 0 || seq >= ctx->desc.max_seqs || layer < 0 || layer >= ctx->layers_stored) return KVD_ERR_INVALID_ARG;
  if (n == 0) return KVD_OK;
  if (!rows || !positions) return KVD_ERR_INVALID_ARG;
  if (!aligned16(rows)) return KVD_ERR_ALIGNMENT;
  int &count = ctx->rows_stored[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
  if (count + n > ctx->desc.max_tokens_per_seq) return KVD_ERR_CAPACITY;
  const size_t slot = store_slot(ctx, layer, seq) + count;
  kvd_status st = launch_checkpoint(ctx, static_cast<const __nv_bfloat16 *>(rows), positions,
                                    ctx->store_rows + slot * ctx->desc.d_hidden * (dtype_bytes(ctx->dtype) / 2), ctx->store_pos + slot,
                                    ctx->store_sumsq + slot, n, ctx->desc.d_hidden, static_cast<cudaStream_t>(stream_));
  if (st == KVD_OK) count += n;
  return st;
}

extern "C" kvd_status kvd_checkpoint_residual_step(kvd_ctx *ctx, int layer, int n, const int32_t *seqs, const void *rows,
                                                   const int32_t *positions, void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (!ctx->store_rows) return KVD_ERR_STATE;
  if (layer < 0 || layer >= ctx->layers_stored) return KVD_ERR_INVALID_ARG;
  if (n == 0) return KVD_OK;
  if (n > KVD_MAX_STORE_RANGES) return KVD_ERR_CAPACITY;
  if (!seqs || !rows || !positions) return KVD_ERR_INVALID_ARG;
  if (!aligned16(rows)) return KVD_ERR_ALIGNMENT;
  // validate everything before any count moves
  std::vector<int> add(ctx->desc.max_seqs, 0);
  CkptSlots slots;
  for (int i = 0; i < n; ++i) {
    const int s = seqs[i];
    if (s < 0 || s >= ctx->desc.max_seqs) return KVD_ERR_INVALID_ARG;
    const int count = ctx->rows_stored[static_cast<size_t>(layer) * ctx->desc.max_seqs + s] + add[s];
    if (count + 1 > ctx->desc.max_tokens_per_seq) return KVD_ERR_CAPACITY;
    slots.slot[i] = static_cast<long long>(store_slot(ctx, layer, s) + count);
    add[s] += 1;
  }
  kvd_status st = launch_checkpoint_scatter(ctx, static_cast<const __nv_bfloat16 *>(rows), positions, slots, n,
                                            ctx->desc.d_hidden, static_cast<cudaStream_t>(stream_));
  if (st == KVD_OK)
    for (int s = 0; s < ctx->desc.max_seqs; ++s) ctx->rows_stored[static_cast<size_t>(layer) * ctx->desc.max_seqs + s] += add[s];
  return st;
}

// The launch parameters every variant of the recompute kernel shares (jobs are filled in by the caller).
static void fill_launch_params(const kvd_ctx *ctx, const LayerState &ls, RecomputeParams &p, int n_jobs, int m_blocks,
                               int k_blocks, int64_t out_row_stride) {
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  p.n_jobs = n_jobs;
  p.num_k_blocks = k_blocks;
  p.num_m_blocks = m_blocks;
  p.num_n_blocks = 2 * kdim / ctx->block_n;
  p.k_cols = kdim;
  p.out_row_stride = out_row_stride;
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
  p.ext_rows = nullptr;
  p.w_scale = nullptr;
  p.rows_out_stride = out_row_stride;
  p.append_n = 0;
  p.append_rows = nullptr;
  p.append_pos = nullptr;
  p.append_sumsq = nullptr;
  p.store_rows = d.max_tokens_per_seq;
  p.row_chunks = d.d_hidden * dtype_bytes(ctx->dtype) / 16;
  // 32-byte stores need every output row 32-byte aligned
  p.wide_store = out_row_stride * dtype_bytes(ctx->dtype) % 32 == 0;
  for (int i = 0; i < n_jobs; ++i)
    if (((reinterpret_cast<uintptr_t>(p.jobs[i].k_out) | reinterpret_cast<uintptr_t>(p.jobs[i].v_out)) & 31u) != 0) p.wide_store = 0;
}

// Shared body of kvd_recompute_kv and kvd_recompute_kv_step: validate, build the job table (store
// ranges first, then the caller's rows), launch once.
// With `fused` (one RcAttend per range, q == nullptr for a range that is to be stored as usual) the
// ranges that carry a query are attended inside the kernel instead of being written.
// `step` (kvd_decode_step_kv): a row stride of their own for the caller rows' outputs and, with append_seqs, the
// rows' STORE_RESIDUAL in the same launch.
struct StepExtra {
  int64_t rows_out_stride;
  const int32_t *append_seqs;  // HOST [n_rows] or nullptr
};
static kvd_status recompute_launch(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                   const void *rows, const int32_t *positions, int n_rows, void *k_rows_out,
                                   void *v_rows_out, int64_t out_row_stride, cudaStream_t stream,
                                   const RcAttend *fused = nullptr, const AttnLaunchHead *fused_head = nullptr,
                                   const StepExtra *step = nullptr) {
  const LayerState &ls = ctx->layers[layer];
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  const int es = dtype_bytes(ctx->dtype);
  if (out_row_stride < kdim) return KVD_ERR_INVALID_ARG;
  if (out_row_stride * es % 16 != 0) return KVD_ERR_ALIGNMENT;
  RecomputeParams p;
  static thread_local FusedParams fp;  // large: keep it off the stack
  int n_jobs = 0, mb = 0;
  bool any_store = false;
  for (int i = 0; i < n_ranges; ++i) {
    const kvd_store_range &r = ranges[i];
    if (r.n < 0) return KVD_ERR_INVALID_ARG;
    if (r.n == 0) continue;
    if (!ctx->store_rows) return KVD_ERR_STATE;
    if (r.seq < 0 || r.seq >= d.max_seqs || layer >= ctx->layers_stored || r.first_row < 0) return KVD_ERR_INVALID_ARG;
    const bool attends = fused && fused[i].q != nullptr;
    if (!attends) {
      if (!r.k_out || !r.v_out) return KVD_ERR_INVALID_ARG;
      if (!aligned16(r.k_out) || !aligned16(r.v_out)) return KVD_ERR_ALIGNMENT;
    }
    if (fused) fp.att[n_jobs] = fused[i];
    const int have = ctx->rows_stored[static_cast<size_t>(layer) * d.max_seqs + r.seq];
    if (r.first_row > have || r.n > have - r.first_row) return KVD_ERR_CAPACITY;
    RcJob &J = p.jobs[n_jobs++];
    J.mb_start = mb;
    J.n = r.n;
    J.row0 = r.first_row;
    J.slab = r.seq;
    J.positions = ctx->store_pos + store_slot(ctx, layer, r.seq) + r.first_row;
    J.sumsq = ctx->store_sumsq + store_slot(ctx, layer, r.seq) + r.first_row;
    J.scale = nullptr;
    J.k_out = static_cast<__nv_bfloat16 *>(r.k_out);
    J.v_out = static_cast<__nv_bfloat16 *>(r.v_out);
    mb += (r.n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);  // 256-row tiles, 128 rows per CTA of a pair
    any_store = true;
  }
  CUtensorMap tmap_rows;
  if (n_rows > 0) {
    if (!rows || !positions || !k_rows_out || !v_rows_out) return KVD_ERR_INVALID_ARG;
    if (!aligned16(rows) || !aligned16(k_rows_out) || !aligned16(v_rows_out)) return KVD_ERR_ALIGNMENT;
    kvd_status st = encode_rows_3d(ctx, &tmap_rows, rows, d.d_hidden, static_cast<uint64_t>(n_rows), 1, es);
    if (st != KVD_OK) return st;
    if (fused) fp.att[n_jobs].q = nullptr;  // the caller's rows are stored
    RcJob &J = p.jobs[n_jobs++];
    J.mb_start = mb;
    J.n = n_rows;
    J.row0 = 0;
    J.slab = -1;
    J.positions = positions;
    J.sumsq = nullptr;
    J.scale = nullptr;
    if (n_rows > RC_INLINE_STAT_ROWS && static_cast<size_t>(n_rows) <= ctx->ext_sumsq_rows) {
      // too many rows for the statistics warps of the main kernel: take the statistics first (same
      // function, same bits).  The scratch is shared by the calls on this context, which are
      // stream-ordered by contract.
      st = launch_rowstats(ctx, static_cast<const __nv_bfloat16 *>(rows), ctx->ext_sumsq, n_rows, d.d_hidden, stream);
      if (st != KVD_OK) return st;
      J.sumsq = ctx->ext_sumsq;
    }
    J.k_out = static_cast<__nv_bfloat16 *>(k_rows_out);
    J.v_out = static_cast<__nv_bfloat16 *>(v_rows_out);
    mb += (n_rows + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);
  }
  if (n_jobs == 0) return KVD_OK;
  // the kernel is handed both maps; an unused one aliases the other
  const CUtensorMap &tmap_store = any_store ? ctx->store_maps[layer] : tmap_rows;
  const CUtensorMap &tmap_ext = n_rows > 0 ? tmap_rows : ctx->store_maps[layer];
  fill_launch_params(ctx, ls, p, n_jobs, mb, d.d_hidden * es / (2 * RC_BLOCK_K), out_row_stride);  // 128 bytes per k block
  p.ext_rows = static_cast<const __nv_bfloat16 *>(rows);
  std::vector<int> add;
  if (step && n_rows > 0) {
    if (step->rows_out_stride < kdim) return KVD_ERR_INVALID_ARG;
    if (step->rows_out_stride * es % 16 != 0) return KVD_ERR_ALIGNMENT;
    p.rows_out_stride = step->rows_out_stride;
    if (step->rows_out_stride * es % 32 != 0) p.wide_store = 0;
    if (step->append_seqs) {
      // STORE_RESIDUAL of the new rows inside this launch: the host assigns the store slots, the statistics
      // warps of the main kernel write rows, positions and sums of squares (everything validated before any count moves)
      if (!ctx->store_rows) return KVD_ERR_STATE;
      if (layer >= ctx->layers_stored) return KVD_ERR_INVALID_ARG;
      if (n_rows > RC_INLINE_STAT_ROWS) return KVD_ERR_CAPACITY;
      add.assign(d.max_seqs, 0);
      for (int i = 0; i < n_rows; ++i) {
        const int sq = step->append_seqs[i];
        if (sq < 0 || sq >= d.max_seqs) return KVD_ERR_INVALID_ARG;
        const int count = ctx->rows_stored[static_cast<size_t>(layer) * d.max_seqs + sq] + add[sq];
        if (count + 1 > d.max_tokens_per_seq) return KVD_ERR_CAPACITY;
        p.append_slot[i] = static_cast<long long>(store_slot(ctx, layer, sq) + count);
        add[sq] += 1;
      }
      p.append_n = n_rows;
      p.append_rows = reinterpret_cast<uint4 *>(ctx->store_rows);
      p.append_pos = ctx->store_pos;
      p.append_sumsq = ctx->store_sumsq;
    }
  }
  if (ctx->trace) {
    const int tiles = p.num_m_blocks * p.num_n_blocks;
    const size_t ctas = 2 * static_cast<size_t>(tiles < ctx->num_sms / 2 ? tiles : ctx->num_sms / 2);
    if (ctas * RC_TRACE_TILES * RC_TRACE_FIELDS * sizeof(long long) <= ctx->trace_bytes) p.trace = ctx->trace;
  }
  if (fused) {
    fp.part_o = fused_head->part_o;
    fp.part_ml = fused_head->part_ml;
    fp.n_q = fused_head->n_q;
    fp.scale_log2e = fused_head->scale_log2e;
    return launch_recompute_fused(ctx, ls, tmap_store, tmap_ext, p, fp, stream);
  }
  kvd_status st = launch_recompute(ctx, ls, tmap_store, tmap_ext, p, stream);
  if (st == KVD_OK && p.append_n > 0)
    for (int sq = 0; sq < d.max_seqs; ++sq) ctx->rows_stored[static_cast<size_t>(layer) * d.max_seqs + sq] += add[sq];
  return st;
}

extern "C" kvd_status kvd_decode_step_kv(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                         int64_t out_row_stride, const void *rows, const int32_t *positions, int n_rows,
                                         const int32_t *append_seqs, void *k_rows_out, void *v_rows_out,
                                         int64_t rows_out_row_stride, void *stream_) {
  if (!ctx || n_ranges < 0 || n_ranges > KVD_MAX_STORE_RANGES || n_rows < 0) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if (!ctx->layers[layer].set) return KVD_ERR_STATE;
  if (n_ranges > 0 && !ranges) return KVD_ERR_INVALID_ARG;
  const int kdim = ctx->desc.n_kv_heads * ctx->desc.d_head;
  StepExtra ex;
  ex.rows_out_stride = rows_out_row_stride > 0 ? rows_out_row_stride : kdim;
  ex.append_seqs = append_seqs;
  return recompute_launch(ctx, layer, ranges, n_ranges, rows, positions, n_rows, k_rows_out, v_rows_out,
                          out_row_stride > 0 ? out_row_stride : kdim, static_cast<cudaStream_t>(stream_), nullptr, nullptr, &ex);
}

// ------------------------------------------------------------------------------ FP8 checkpoints
extern "C" size_t kvd_store_bytes_fp8(const kvd_model_desc *d, int layers_stored) {
  if (check_desc(d) != KVD_OK || layers_stored <= 0 || d->d_hidden % 16 != 0) return 0;
  const size_t slots = static_cast<size_t>(layers_stored) * d->max_seqs * d->max_tokens_per_seq;
  // codes, then positions, sums of squares and scales, each region starting at a 256-byte multiple
  return round_up(slots * d->d_hidden, 256) + 3 * round_up(slots * 4, 256);
}

extern "C" kvd_status kvd_attach_store_fp8(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored) {
  if (!ctx || !arena || layers_stored <= 0 || layers_stored > ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return KVD_ERR_ALIGNMENT;
  const size_t need = kvd_store_bytes_fp8(&ctx->desc, layers_stored);
  if (need == 0) return KVD_ERR_SHAPE;
  if (bytes < need) return KVD_ERR_CAPACITY;
  const kvd_model_desc &d = ctx->desc;
  const size_t slots = static_cast<size_t>(layers_stored) * d.max_seqs * d.max_tokens_per_seq;
  uint8_t *base = static_cast<uint8_t *>(arena);
  ctx->store8_codes = base;
  ctx->store8_pos = reinterpret_cast<int32_t *>(base + round_up(slots * d.d_hidden, 256));
  ctx->store8_sumsq = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(ctx->store8_pos) + round_up(slots * 4, 256));
  ctx->store8_scale = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(ctx->store8_sumsq) + round_up(slots * 4, 256));
  ctx->layers_stored8 = layers_stored;
  ctx->rows_stored8.assign(static_cast<size_t>(layers_stored) * d.max_seqs, 0);
  ctx->store8_maps.resize(layers_stored);
  for (int l = 0; l < layers_stored; ++l) {
    const uint8_t *lb = ctx->store8_codes + static_cast<size_t>(l) * d.max_seqs * d.max_tokens_per_seq * d.d_hidden;
    kvd_status st = encode_rows_3d(ctx, &ctx->store8_maps[l], lb, d.d_hidden, d.max_tokens_per_seq, d.max_seqs, 1);
    if (st != KVD_OK) {
      ctx->store8_codes = nullptr;
      ctx->layers_stored8 = 0;
      return st;
    }
  }
  return KVD_OK;
}

extern "C" int kvd_rows_stored_fp8(const kvd_ctx *ctx, int layer, int seq) {
  if (!ctx || !ctx->store8_codes || layer < 0 || layer >= ctx->layers_stored8 || seq < 0 || seq >= ctx->desc.max_seqs)
    return -1;
  return ctx->rows_stored8[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
}

extern "C" kvd_status kvd_checkpoint_residual_fp8(kvd_ctx *ctx, int seq, int layer, const void *rows,
                                                  const int32_t *positions, int n, void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (!ctx->store8_codes) return KVD_ERR_STATE;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;  // the quantiser reads bf16 rows
  if (seq < 0 || seq >= ctx->desc.max_seqs || layer < 0 || layer >= ctx->layers_stored8) return KVD_ERR_INVALID_ARG;
  if (n == 0) return KVD_OK;
  if (!rows || !positions) return KVD_ERR_INVALID_ARG;
  if (!aligned16(rows)) return KVD_ERR_ALIGNMENT;
  int &count = ctx->rows_stored8[static_cast<size_t>(layer) * ctx->desc.max_seqs + seq];
  if (count + n > ctx->desc.max_tokens_per_seq) return KVD_ERR_CAPACITY;
  const size_t slot = store_slot(ctx, layer, seq) + count;
  kvd_status st = launch_checkpoint_fp8(ctx, static_cast<const __nv_bfloat16 *>(rows), positions,
                                        ctx->store8_codes + slot * ctx->desc.d_hidden, ctx->store8_pos + slot,
                                        ctx->store8_sumsq + slot, ctx->store8_scale + slot, n, ctx->desc.d_hidden,
                                        static_cast<cudaStream_t>(stream_));
  if (st == KVD_OK) count += n;
  return st;
}

// Shared body of kvd_recompute_kv_fp8 and kvd_decode_attention_recompute_fp8: validate, build the
// job table from ranges of the FP8 store, launch once.  With `fused` (one RcAttend per range, q ==
// nullptr for a range whose K/V are written) the ranges that carry a query are attended in the kernel.
static kvd_status recompute_launch_fp8(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                       const kvd_fp8_rows *rows, int64_t out_row_stride, cudaStream_t stream,
                                       const RcAttend *fused = nullptr, const AttnLaunchHead *fused_head = nullptr) {
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set || !ls.wt8) return KVD_ERR_STATE;
  bool any_range = false;
  for (int i = 0; i < n_ranges; ++i) any_range |= ranges[i].n > 0;
  if (any_range && (!ctx->store8_codes || layer >= ctx->layers_stored8)) return ctx->store8_codes ? KVD_ERR_INVALID_ARG : KVD_ERR_STATE;
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  if (out_row_stride < kdim) return KVD_ERR_INVALID_ARG;
  if (out_row_stride % 8 != 0) return KVD_ERR_ALIGNMENT;
  RecomputeParams p;
  static thread_local FusedParams fp;  // large: keep it off the stack
  int n_jobs = 0, mb = 0;
  for (int i = 0; i < n_ranges; ++i) {
    const kvd_store_range &r = ranges[i];
    if (r.n < 0) return KVD_ERR_INVALID_ARG;
    if (r.n == 0) continue;
    if (r.seq < 0 || r.seq >= d.max_seqs || r.first_row < 0) return KVD_ERR_INVALID_ARG;
    const bool attends = fused && fused[i].q != nullptr;
    if (!attends) {
      if (!r.k_out || !r.v_out) return KVD_ERR_INVALID_ARG;
      if (!aligned16(r.k_out) || !aligned16(r.v_out)) return KVD_ERR_ALIGNMENT;
    }
    if (fused) fp.att[n_jobs] = fused[i];
    const int have = ctx->rows_stored8[static_cast<size_t>(layer) * d.max_seqs + r.seq];
    if (r.first_row > have || r.n > have - r.first_row) return KVD_ERR_CAPACITY;
    const size_t slot = store_slot(ctx, layer, r.seq) + r.first_row;
    RcJob &J = p.jobs[n_jobs++];
    J.mb_start = mb;
    J.n = r.n;
    J.row0 = r.first_row;
    J.slab = r.seq;
    J.positions = ctx->store8_pos + slot;
    J.sumsq = ctx->store8_sumsq + slot;
    J.scale = ctx->store8_scale + slot;
    J.k_out = static_cast<__nv_bfloat16 *>(r.k_out);
    J.v_out = static_cast<__nv_bfloat16 *>(r.v_out);
    mb += (r.n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);
  }
  // the caller's own quantised rows (kvd_quantize_rows_fp8): one more job, always stored
  CUtensorMap tmap_rows;
  const bool have_rows = rows != nullptr && rows->n > 0;
  if (rows != nullptr && rows->n < 0) return KVD_ERR_INVALID_ARG;
  if (have_rows) {
    if (!rows->codes || !rows->scales || !rows->sumsq || !rows->positions || !rows->k_out || !rows->v_out) return KVD_ERR_INVALID_ARG;
    if (!aligned16(rows->codes) || !aligned16(rows->k_out) || !aligned16(rows->v_out)) return KVD_ERR_ALIGNMENT;
    kvd_status st = encode_rows_3d(ctx, &tmap_rows, rows->codes, d.d_hidden, static_cast<uint64_t>(rows->n), 1, 1);
    if (st != KVD_OK) return st;
    if (fused) fp.att[n_jobs] = RcAttend{};
    RcJob &J = p.jobs[n_jobs++];
    J.mb_start = mb;
    J.n = rows->n;
    J.row0 = 0;
    J.slab = -1;
    J.positions = rows->positions;
    J.sumsq = rows->sumsq;
    J.scale = rows->scales;
    J.k_out = static_cast<__nv_bfloat16 *>(rows->k_out);
    J.v_out = static_cast<__nv_bfloat16 *>(rows->v_out);
    mb += (rows->n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);
  }
  if (n_jobs == 0) return KVD_OK;
  // the kernel is handed both maps; an unused one aliases the other
  const bool any_store = n_jobs > (have_rows ? 1 : 0);
  const CUtensorMap &map_store = any_store ? ctx->store8_maps[layer] : tmap_rows;
  const CUtensorMap &map_rows = have_rows ? tmap_rows : ctx->store8_maps[layer];
  // 128 channels per k block; the tail reads zeros
  fill_launch_params(ctx, ls, p, n_jobs, mb, (d.d_hidden + 2 * RC_BLOCK_K - 1) / (2 * RC_BLOCK_K), out_row_stride);
  p.w_scale = ls.w_scale8;
  if (ctx->trace) {
    const int tiles = p.num_m_blocks * p.num_n_blocks;
    const size_t ctas = 2 * static_cast<size_t>(tiles < ctx->num_sms / 2 ? tiles : ctx->num_sms / 2);
    if (ctas * RC_TRACE_TILES * RC_TRACE_FIELDS * sizeof(long long) <= ctx->trace_bytes) p.trace = ctx->trace;
  }
  if (fused) {
    fp.part_o = fused_head->part_o;
    fp.part_ml = fused_head->part_ml;
    fp.n_q = fused_head->n_q;
    fp.scale_log2e = fused_head->scale_log2e;
    return launch_recompute_fused(ctx, ls, map_store, map_rows, p, fp, stream, 1);
  }
  return launch_recompute_fp8(ctx, ls, map_store, map_rows, p, stream);
}

extern "C" kvd_status kvd_quantize_rows_fp8(kvd_ctx *ctx, const void *rows, int n, void *codes_out, float *scales_out,
                                            float *sumsq_out, void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  if (ctx->desc.d_hidden % 16 != 0) return KVD_ERR_SHAPE;
  if (n == 0) return KVD_OK;
  if (!rows || !codes_out || !scales_out || !sumsq_out) return KVD_ERR_INVALID_ARG;
  if (!aligned16(rows) || !aligned16(codes_out)) return KVD_ERR_ALIGNMENT;
  return launch_checkpoint_fp8(ctx, static_cast<const __nv_bfloat16 *>(rows), nullptr, static_cast<uint8_t *>(codes_out),
                               nullptr, sumsq_out, scales_out, n, ctx->desc.d_hidden, static_cast<cudaStream_t>(stream_));
}

extern "C" kvd_status kvd_recompute_kv_fp8_rows(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                                const kvd_fp8_rows *rows, int64_t out_row_stride, void *stream_) {
  if (!ctx || n_ranges < 0 || n_ranges > KVD_MAX_STORE_RANGES || (n_ranges > 0 && !ranges)) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  return recompute_launch_fp8(ctx, layer, ranges, n_ranges, rows, out_row_stride, static_cast<cudaStream_t>(stream_));
}

extern "C" kvd_status kvd_recompute_kv_fp8(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                           int64_t out_row_stride, void *stream_) {
  if (!ctx || n_ranges < 0 || n_ranges > KVD_MAX_STORE_RANGES || (n_ranges > 0 && !ranges)) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  return recompute_launch_fp8(ctx, layer, ranges, n_ranges, nullptr, out_row_stride, static_cast<cudaStream_t>(stream_));
}

extern "C" kvd_status kvd_recompute_kv(kvd_ctx *ctx, int layer, const void *rows, const int32_t *positions, int n,
                                       int seq, int first_row, void *k_out, void *v_out, int64_t out_row_stride,
                                       void *stream_) {
  if (!ctx || n < 0) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if (!ctx->layers[layer].set) return KVD_ERR_STATE;
  if (n == 0) return KVD_OK;
  if (!k_out || !v_out) return KVD_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (rows) {
    if (!positions) return KVD_ERR_INVALID_ARG;
    return recompute_launch(ctx, layer, nullptr, 0, rows, positions, n, k_out, v_out, out_row_stride, stream);
  }
  if (positions) return KVD_ERR_INVALID_ARG;
  if (!ctx->store_rows) return KVD_ERR_STATE;
  kvd_store_range r;
  r.seq = seq;
  r.first_row = first_row;
  r.n = n;
  r.reserved = 0;
  r.k_out = k_out;
  r.v_out = v_out;
  return recompute_launch(ctx, layer, &r, 1, nullptr, nullptr, 0, nullptr, nullptr, out_row_stride, stream);
}

extern "C" kvd_status kvd_recompute_kv_step(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                            const void *rows, const int32_t *positions, int n_rows, void *k_rows_out,
                                            void *v_rows_out, int64_t out_row_stride, void *stream_) {
  if (!ctx || n_ranges < 0 || n_rows < 0) return KVD_ERR_INVALID_ARG;
  if (n_ranges > KVD_MAX_STORE_RANGES || (n_ranges > 0 && !ranges)) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  if (!ctx->layers[layer].set) return KVD_ERR_STATE;
  return recompute_launch(ctx, layer, ranges, n_ranges, rows, positions, n_rows, k_rows_out, v_rows_out, out_row_stride,
                          static_cast<cudaStream_t>(stream_));
}

// Validate the segments of `batch` sequences (nothing is launched on an error).
static kvd_status check_segments(const kvd_ctx *ctx, int batch, const int32_t *q_pos, const kvd_kv_segment *segs,
                                 int n_segs) {
  const kvd_model_desc &d = ctx->desc;
  const int kdim = d.n_kv_heads * d.d_head;
  for (int b = 0; b < batch; ++b) {
    if (q_pos[b] < 0) return KVD_ERR_INVALID_ARG;
    for (int s = 0; s < n_segs; ++s) {
      const kvd_kv_segment &sg = segs[static_cast<size_t>(b) * n_segs + s];
      if (sg.len < 0 || sg.first_pos < 0) return KVD_ERR_INVALID_ARG;
      if (sg.len == 0) continue;
      if (!sg.k || !sg.v || sg.row_stride < kdim) return KVD_ERR_INVALID_ARG;
      if (!aligned16(sg.k) || !aligned16(sg.v) || sg.row_stride % 8 != 0) return KVD_ERR_ALIGNMENT;
      if (static_cast<int64_t>(sg.first_pos) + sg.len > INT32_MAX) return KVD_ERR_INVALID_ARG;
      for (int s2 = 0; s2 < s; ++s2) {
        const kvd_kv_segment &o = segs[static_cast<size_t>(b) * n_segs + s2];
        if (o.len == 0) continue;
        if (sg.first_pos < o.first_pos + o.len && o.first_pos < sg.first_pos + sg.len) return KVD_ERR_INVALID_ARG;
      }
    }
  }
  return KVD_OK;
}

// Describe one launch over sequences b0 .. b0 + nb - 1 (nb <= AT_MAX_SEQS): segments, visible range, the
// split into chunks and the slots of the partial arrays.  pre_parts[b] (may be NULL) slots are left
// in front of a sequence's chunks for partials that another kernel writes (fused recompute); the
// merge kernel combines them with the chunks, in slot order.
static kvd_status build_attn_launch(kvd_ctx *ctx, const LayerState &ls, int b0, int nb, const void *q,
                                    const int32_t *q_pos, const kvd_kv_segment *segs, int n_segs, float scale,
                                    void *out, const int *pre_parts, AttnLaunch &L) {
  const kvd_model_desc &d = ctx->desc;
  int parts = 0, slots = 0;
  for (int i = 0; i < nb; ++i) {
    const int b = b0 + i;
    AttnSeq &S = L.seq[i];
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
    int lo = ls.window > 0 ? S.q_pos - ls.window + 1 : 0;
    if (lo < 0) lo = 0;
    if (min_first > lo) lo = min_first;
    int hi = S.q_pos < max_last ? S.q_pos : max_last;
    S.lo_pos = lo;
    S.hi_pos = hi;
    S.part_base = parts;
    if (max_last < 0 || hi < lo) {
      S.n_chunks = 0;
      S.iters = 1;
      S.chunk0_pos = 0;
    } else {
      // the split depends on the visible position range only
      S.iters = attn_iters_for_span(d.d_head, d.n_kv_heads, hi - lo + 1);
      const int ck = attn_chunk_keys(d.d_head, S.iters);
      S.chunk0_pos = lo / ck * ck;
      S.n_chunks = hi / ck - lo / ck + 1;
    }
    const int pre = pre_parts ? pre_parts[b] : 0;
    S.merge_base = slots;
    S.slot_base = slots + pre;
    S.merge_count = pre + S.n_chunks;
    slots += S.merge_count;
    parts += S.n_chunks;
  }
  if (slots > ctx->max_parts) return KVD_ERR_CAPACITY;
  const float sc = scale > 0.f ? scale : 1.0f / sqrtf(static_cast<float>(d.d_head));
  L.n_seqs = nb;
  L.total_chunks = parts;
  L.n_q = d.n_q_heads;
  L.n_kv = d.n_kv_heads;
  L.q = static_cast<const __nv_bfloat16 *>(q) + static_cast<size_t>(b0) * d.n_q_heads * d.d_head;
  L.out = static_cast<__nv_bfloat16 *>(out) + static_cast<size_t>(b0) * d.n_q_heads * d.d_head;
  L.part_o = ctx->part_o;
  L.part_ml = ctx->part_ml;
  L.status = ctx->d_status;
  L.max_parts = ctx->max_parts;
  L.scale_log2e = sc * 1.4426950408889634f;
  return KVD_OK;
}

extern "C" kvd_status kvd_decode_attention(kvd_ctx *ctx, int layer, int batch, const void *q, const int32_t *q_pos,
                                           const kvd_kv_segment *segs, int n_segs, float scale, void *out,
                                           void *stream_) {
  if (!ctx || batch < 0 || n_segs < 0 || n_segs > KVD_MAX_SEGMENTS) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (!ctx->part_o) return KVD_ERR_STATE;
  if (ctx->dtype == KVD_DTYPE_F32) return KVD_ERR_UNSUPPORTED;  // attention reads 16-bit K/V
  if (batch == 0) return KVD_OK;
  if (!q || !q_pos || !out || (n_segs > 0 && !segs)) return KVD_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return KVD_ERR_ALIGNMENT;
  const kvd_model_desc &d = ctx->desc;
  if (batch > d.max_batch) return KVD_ERR_CAPACITY;
  const int group = d.n_q_heads / d.n_kv_heads;
  kvd_status st = check_segments(ctx, batch, q_pos, segs, n_segs);
  if (st != KVD_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  static thread_local AttnLaunch L;  // large: keep it off the stack
  for (int b0 = 0; b0 < batch; b0 += AT_MAX_SEQS) {
    const int nb = batch - b0 < AT_MAX_SEQS ? batch - b0 : AT_MAX_SEQS;
    st = build_attn_launch(ctx, ls, b0, nb, q, q_pos, segs, n_segs, scale, out, nullptr, L);
    if (st != KVD_OK) return st;
    // sequences without a visible key stream nothing; the merge kernel writes their zeros
    st = launch_attention(ctx, L, d.d_head, group, stream);
    if (st != KVD_OK) return st;
  }
  return KVD_OK;
}

extern "C" int kvd_fused_recompute_pays(const kvd_model_desc *desc, int64_t total_rows, int fp8) {
  if (check_desc(desc) != KVD_OK || total_rows <= 0) return 0;
  const int group = desc->n_q_heads / desc->n_kv_heads, kdim = desc->n_kv_heads * desc->d_head;
  // the shapes the fused kernel exists for
  if (pick_block_n(desc) != 256 || kdim % 256 != 0 ||
      !((desc->d_head == 256 && (group == 1 || group == 2)) || (desc->d_head == 128 && (group == 1 || group == 2 || group == 4))))
    return 0;
  return total_rows >= (fp8 ? 4096 : 16384) ? 1 : 0;
}

extern "C" kvd_status kvd_decode_attention_rows(kvd_ctx *ctx, int layer, int n_rows, const void *q, const int32_t *q_pos,
                                                const kvd_kv_segment *segs, int n_segs, float scale, void *out,
                                                void *stream_) {
  if (!ctx || n_rows < 0 || n_segs < 0 || n_segs > KVD_MAX_SEGMENTS) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (!ctx->part_o) return KVD_ERR_STATE;
  if (ctx->dtype == KVD_DTYPE_F32) return KVD_ERR_UNSUPPORTED;
  if (n_rows == 0) return KVD_OK;
  if (!q || !q_pos || !out || (n_segs > 0 && !segs)) return KVD_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return KVD_ERR_ALIGNMENT;
  const kvd_model_desc &d = ctx->desc;
  const int group = d.n_q_heads / d.n_kv_heads;
  // the one sequence's segments, validated once with a query position that every row's replaces below
  int32_t zero = 0;
  kvd_status st = check_segments(ctx, 1, &zero, segs, n_segs);
  if (st != KVD_OK) return st;
  for (int i = 0; i < n_rows; ++i)
    if (q_pos[i] < 0) return KVD_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  static thread_local AttnLaunch L;  // large: keep it off the stack
  // every row is a "sequence" of a decode-attention launch that shares the segments; a launch takes as many
  // rows as the launch descriptor (AT_MAX_SEQS) and the workspace's partial slots (max_parts) hold
  std::vector<kvd_kv_segment> rep(static_cast<size_t>(AT_MAX_SEQS) * (n_segs > 0 ? n_segs : 1));
  for (int i = 0; i < AT_MAX_SEQS; ++i)
    for (int sg = 0; sg < n_segs; ++sg) rep[static_cast<size_t>(i) * n_segs + sg] = segs[sg];
  const size_t row_elems = static_cast<size_t>(d.n_q_heads) * d.d_head;
  const int es = 2;  // bf16 or fp16 queries and outputs
  int r0 = 0;
  while (r0 < n_rows) {
    int nb = n_rows - r0 < AT_MAX_SEQS ? n_rows - r0 : AT_MAX_SEQS;
    const uint8_t *qb = static_cast<const uint8_t *>(q) + static_cast<size_t>(r0) * row_elems * es;
    uint8_t *ob = static_cast<uint8_t *>(out) + static_cast<size_t>(r0) * row_elems * es;
    // shrink the launch until its partials fit the workspace (one row always has to)
    while (true) {
      st = build_attn_launch(ctx, ls, 0, nb, qb, q_pos + r0, rep.data(), n_segs, scale, ob, nullptr, L);
      if (st != KVD_ERR_CAPACITY || nb == 1) break;
      nb = nb / 2;
    }
    if (st != KVD_OK) return st;
    st = launch_attention(ctx, L, d.d_head, group, stream);
    if (st != KVD_OK) return st;
    r0 += nb;
  }
  return KVD_OK;
}

// Decode attention over [K/V recomputed from store ranges] + [live segments], the recomputed part
// inside the recompute kernel (its K/V never reach memory); see kvd.h.
extern "C" kvd_status kvd_decode_attention_recompute(kvd_ctx *ctx, int layer, int batch, const void *q,
                                                     const int32_t *q_pos, const kvd_store_range *ranges,
                                                     const void *rows, const int32_t *positions, int n_rows,
                                                     void *k_rows_out, void *v_rows_out, int64_t out_row_stride,
                                                     const kvd_kv_segment *segs, int n_segs, float scale,
                                                     void *out, void *stream_) {
  if (!ctx || batch < 0 || n_segs < 0 || n_segs > KVD_MAX_SEGMENTS || n_rows < 0) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (!ctx->part_o || !ctx->store_rows) return KVD_ERR_STATE;
  if (ctx->dtype == KVD_DTYPE_F32) return KVD_ERR_UNSUPPORTED;  // bf16 and fp16 contexts
  const kvd_model_desc &d = ctx->desc;
  const int group = d.n_q_heads / d.n_kv_heads, kdim = d.n_kv_heads * d.d_head;
  // shapes the fused kernel is built for (nothing is launched otherwise)
  if (ctx->block_n != 256 || kdim % 256 != 0 || !((d.d_head == 256 && (group == 1 || group == 2)) ||
                                                   (d.d_head == 128 && (group == 1 || group == 2 || group == 4))))
    return KVD_ERR_UNSUPPORTED;
  if (batch == 0 && n_rows == 0) return KVD_OK;
  if (batch > 0 && (!q || !q_pos || !out || !ranges || (n_segs > 0 && !segs))) return KVD_ERR_INVALID_ARG;
  if (batch > 0 && (!aligned16(q) || !aligned16(out))) return KVD_ERR_ALIGNMENT;
  if (batch > d.max_batch || batch > KVD_MAX_STORE_RANGES) return KVD_ERR_CAPACITY;
  kvd_status st = check_segments(ctx, batch, q_pos, segs, n_segs);
  if (st != KVD_OK) return st;
  int pre[KVD_MAX_STORE_RANGES];
  for (int b = 0; b < batch; ++b) {
    if (ranges[b].n < 0) return KVD_ERR_INVALID_ARG;
    pre[b] = (ranges[b].n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);  // one partial per 256-row block
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  static thread_local AttnLaunch L;  // large: keep it off the stack
  st = build_attn_launch(ctx, ls, 0, batch, q, q_pos, segs, n_segs, scale, out, pre, L);
  if (st != KVD_OK) return st;
  RcAttend att[KVD_MAX_STORE_RANGES];
  for (int b = 0; b < batch; ++b) {
    att[b].q = static_cast<const __nv_bfloat16 *>(q) + static_cast<size_t>(b) * d.n_q_heads * d.d_head;
    att[b].q_pos = q_pos[b];
    att[b].lo_pos = ls.window > 0 && q_pos[b] - ls.window + 1 > 0 ? q_pos[b] - ls.window + 1 : 0;
    att[b].part_base = L.seq[b].merge_base;
    att[b].reserved = 0;
  }
  st = recompute_launch(ctx, layer, ranges, batch, rows, positions, n_rows, k_rows_out, v_rows_out,
                        out_row_stride > 0 ? out_row_stride : kdim, stream, att, &L);
  if (st != KVD_OK) return st;
  if (batch == 0) return KVD_OK;
  return launch_attention(ctx, L, d.d_head, group, stream);
}

// The same over the FP8 store: ranges[b] is attended by query b; store_ranges and the caller's quantised rows
// are written as K/V.
extern "C" kvd_status kvd_decode_attention_recompute_fp8_rows(kvd_ctx *ctx, int layer, int batch, const void *q,
                                                              const int32_t *q_pos, const kvd_store_range *ranges,
                                                              const kvd_store_range *store_ranges, int n_store_ranges,
                                                              const kvd_fp8_rows *rows, int64_t out_row_stride,
                                                              const kvd_kv_segment *segs, int n_segs, float scale,
                                                              void *out, void *stream_) {
  if (!ctx || batch < 0 || n_segs < 0 || n_segs > KVD_MAX_SEGMENTS || n_store_ranges < 0) return KVD_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->desc.n_layers) return KVD_ERR_INVALID_ARG;
  const LayerState &ls = ctx->layers[layer];
  if (!ls.set) return KVD_ERR_STATE;
  if (!ctx->part_o || !ctx->store8_codes || !ls.wt8) return KVD_ERR_STATE;
  if (ctx->dtype != KVD_DTYPE_BF16) return KVD_ERR_UNSUPPORTED;
  const kvd_model_desc &d = ctx->desc;
  const int group = d.n_q_heads / d.n_kv_heads, kdim = d.n_kv_heads * d.d_head;
  if (ctx->block_n != 256 || kdim % 256 != 0 || !((d.d_head == 256 && (group == 1 || group == 2)) ||
                                                   (d.d_head == 128 && (group == 1 || group == 2 || group == 4))))
    return KVD_ERR_UNSUPPORTED;
  if (batch == 0 && n_store_ranges == 0 && (rows == nullptr || rows->n == 0)) return KVD_OK;
  if (batch > 0 && (!q || !q_pos || !out || !ranges || (n_segs > 0 && !segs))) return KVD_ERR_INVALID_ARG;
  if (n_store_ranges > 0 && !store_ranges) return KVD_ERR_INVALID_ARG;
  if (batch > 0 && (!aligned16(q) || !aligned16(out))) return KVD_ERR_ALIGNMENT;
  if (batch > d.max_batch || batch + n_store_ranges > KVD_MAX_STORE_RANGES) return KVD_ERR_CAPACITY;
  kvd_status st = check_segments(ctx, batch, q_pos, segs, n_segs);
  if (st != KVD_OK) return st;
  int pre[KVD_MAX_STORE_RANGES];
  for (int b = 0; b < batch; ++b) {
    if (ranges[b].n < 0) return KVD_ERR_INVALID_ARG;
    pre[b] = (ranges[b].n + 2 * RC_BLOCK_M - 1) / (2 * RC_BLOCK_M);  // one partial per 256-row block
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  static thread_local AttnLaunch L;  // large: keep it off the stack
  st = build_attn_launch(ctx, ls, 0, batch, q, q_pos, segs, n_segs, scale, out, pre, L);
  if (st != KVD_OK) return st;
  kvd_store_range all[KVD_MAX_STORE_RANGES];
  RcAttend att[KVD_MAX_STORE_RANGES];
  for (int b = 0; b < batch; ++b) {
    all[b] = ranges[b];
    att[b].q = static_cast<const __nv_bfloat16 *>(q) + static_cast<size_t>(b) * d.n_q_heads * d.d_head;
    att[b].q_pos = q_pos[b];
    att[b].lo_pos = ls.window > 0 && q_pos[b] - ls.window + 1 > 0 ? q_pos[b] - ls.window + 1 : 0;
    att[b].part_base = L.seq[b].merge_base;
    att[b].reserved = 0;
  }
  for (int i = 0; i < n_store_ranges; ++i) {
    all[batch + i] = store_ranges[i];
    att[batch + i] = RcAttend{};
  }
  st = recompute_launch_fp8(ctx, layer, all, batch + n_store_ranges, rows, out_row_stride > 0 ? out_row_stride : kdim,
                            stream, att, &L);
  if (st != KVD_OK) return st;
  if (batch == 0) return KVD_OK;
  return launch_attention(ctx, L, d.d_head, group, stream);
}

extern "C" kvd_status kvd_decode_attention_recompute_fp8(kvd_ctx *ctx, int layer, int batch, const void *q,
                                                         const int32_t *q_pos, const kvd_store_range *ranges,
                                                         const kvd_store_range *store_ranges, int n_store_ranges,
                                                         int64_t out_row_stride, const kvd_kv_segment *segs,
                                                         int n_segs, float scale, void *out, void *stream_) {
  return kvd_decode_attention_recompute_fp8_rows(ctx, layer, batch, q, q_pos, ranges, store_ranges, n_store_ranges, nullptr,
                                                 out_row_stride, segs, n_segs, scale, out, stream_);
}

extern "C" kvd_status kvd_memory_stats(const kvd_ctx *ctx, kvd_mem_stats *out) {
  if (!ctx || !out) return KVD_ERR_INVALID_ARG;
  const kvd_model_desc &d = ctx->desc;
  memset(out, 0, sizeof(*out));
  uint64_t rows_total = 0, tokens = 0;
  for (int l = 0; l < ctx->layers_stored; ++l) {
    uint64_t layer_rows = 0;
    for (int s = 0; s < d.max_seqs; ++s) layer_rows += ctx->rows_stored[static_cast<size_t>(l) * d.max_seqs + s];
    rows_total += layer_rows;
    if (layer_rows > tokens) tokens = layer_rows;
  }
  out->checkpoint_bytes_used = rows_total * (static_cast<uint64_t>(d.d_hidden) * dtype_bytes(ctx->dtype) + 8);  // row, position, sum of squares
  out->checkpoint_bytes_capacity = ctx->layers_stored > 0 ? kvd_store_bytes_dtype(&d, ctx->layers_stored, ctx->dtype) : 0;
  // the FP8 store counts too: codes, position, sum of squares, scale
  uint64_t rows8 = 0;
  for (int l = 0; l < ctx->layers_stored8; ++l) {
    uint64_t layer_rows = 0;
    for (int s = 0; s < d.max_seqs; ++s) layer_rows += ctx->rows_stored8[static_cast<size_t>(l) * d.max_seqs + s];
    rows8 += layer_rows;
    if (layer_rows > tokens) tokens = layer_rows;
  }
  out->checkpoint_bytes_used += rows8 * (static_cast<uint64_t>(d.d_hidden) + 12);
  out->checkpoint_bytes_capacity += ctx->layers_stored8 > 0 ? kvd_store_bytes_fp8(&d, ctx->layers_stored8) : 0;
  // ... and the FP4 store: codes, block scales, position, sum of squares, row scale
  uint64_t rows4 = 0;
  for (int l = 0; l < ctx->layers_stored4; ++l) {
    uint64_t layer_rows = 0;
    for (int s = 0; s < d.max_seqs; ++s) layer_rows += ctx->rows_stored4[static_cast<size_t>(l) * d.max_seqs + s];
    rows4 += layer_rows;
    if (layer_rows > tokens) tokens = layer_rows;
  }
  out->checkpoint_bytes_used += rows4 * (static_cast<uint64_t>(d.d_hidden) / 2 + d.d_hidden / 16 + 12);
  out->checkpoint_bytes_capacity += ctx->layers_stored4 > 0 ? kvd_store_bytes_fp4(&d, ctx->layers_stored4) : 0;
  out->workspace_bytes = ctx->workspace_bytes;
  out->prepared_weight_bytes = ctx->prepared_bytes;
  out->tokens_stored = tokens;
  out->eq23_kv_bytes_per_token = 2ull * d.n_layers * d.n_kv_heads * d.d_head * dtype_bytes(ctx->dtype);
  out->eq24_residual_bytes_per_token = static_cast<uint64_t>(d.d_hidden) * dtype_bytes(ctx->dtype);
  out->per_layer_residual_bytes_per_token = static_cast<uint64_t>(d.n_layers) * d.d_hidden * dtype_bytes(ctx->dtype);
  return KVD_OK;
}

extern "C" kvd_status kvd_poll_status(kvd_ctx *ctx, void *stream_) {
  if (!ctx) return KVD_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  cudaError_t e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "kvd_poll_status sync");
  int word = 0;
  e = cudaMemcpy(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "kvd_poll_status read");
  if (word != 0) {
    e = cudaMemset(ctx->d_status, 0, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "kvd_poll_status clear");
  }
  if (word & STATUS_TIMEOUT) return KVD_ERR_TIMEOUT;
  if (word & STATUS_BOUNDS) return KVD_ERR_BOUNDS;
  if (word & STATUS_POSITION) return KVD_ERR_POSITION;
  return KVD_OK;
}

extern "C" int kvd_build_has_checks(void) {
#ifdef KVD_CHECK
  return 1;
#else
  return 0;
#endif
}

extern "C" kvd_status kvd_selftest_bounds_check(kvd_ctx *ctx, void *stream_) {
  if (!ctx) return KVD_ERR_INVALID_ARG;
  return launch_selftest_bounds(ctx, static_cast<cudaStream_t>(stream_));
}

extern "C" kvd_status kvd_selftest_wait_timeout(kvd_ctx *ctx, int limit_ms, void *stream_) {
  if (!ctx || limit_ms <= 0 || limit_ms > 1000) return KVD_ERR_INVALID_ARG;
  return launch_selftest_timeout(ctx, static_cast<unsigned long long>(limit_ms) * 1000000ull,
                                 static_cast<cudaStream_t>(stream_));
}

extern "C" kvd_status kvd_set_trace(kvd_ctx *ctx, void *buf, size_t bytes) {
  if (!ctx) return KVD_ERR_INVALID_ARG;
  if (buf && (reinterpret_cast<uintptr_t>(buf) & 7u) != 0) return KVD_ERR_ALIGNMENT;
  ctx->trace = static_cast<long long *>(buf);
  ctx->trace_bytes = buf ? bytes : 0;
  return KVD_OK;
}

extern "C" uint64_t kvd_launch_count(const kvd_ctx *ctx) { return ctx ? ctx->launches : 0; }

extern "C" const char *kvd_last_cuda_error(const kvd_ctx *ctx) { return ctx ? ctx->last_error.c_str() : ""; }
