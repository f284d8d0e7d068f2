// Host-side context and the parameter blocks passed to the kernels.  Internal to the library.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include <map>
#include <string>
#include <vector>

#include "../../include/kvd.h"

namespace kvd {

// device status word bits (written by kernels with atomicOr, read by kvd_poll_status)
constexpr int STATUS_TIMEOUT = 1;
constexpr int STATUS_POSITION = 2;
constexpr int STATUS_BOUNDS = 4;  // checking build: an index test failed (the access was skipped)

// Index tests of the checking build (-DKVD_CHECK): `if (KVD_BOUNDS_OK(cond, status)) access;`.  A failed test
// records STATUS_BOUNDS and yields false, so the access is skipped; the release build compiles the test away.
#ifdef KVD_CHECK
#define KVD_BOUNDS_OK(cond, status) ((cond) ? true : ((status) != nullptr ? (atomicOr((status), kvd::STATUS_BOUNDS), false) : false))
#else
#define KVD_BOUNDS_OK(cond, status) (true)
#endif

constexpr int ROPE_LO_BITS = 4;  // position = hi * 16 + lo; one table per part
constexpr int ROPE_LO_SIZE = 1 << ROPE_LO_BITS;

// ------------------------------------------------------------------------------ recompute GEMM
constexpr int RC_BLOCK_M = 128;
constexpr int RC_BLOCK_K = 64;
// caller rows up to this count have their statistics taken inside the recompute kernel (its four
// statistics warps cover them under the main loop of one tile pair); more rows get a kernel of their own
constexpr int RC_INLINE_STAT_ROWS = 64;
constexpr int RC_TRACE_TILES = 8;    // tiles per CTA recorded when a trace buffer is attached
constexpr int RC_TRACE_FIELDS = 16;  // int64 slots per (CTA, tile); see kvd_set_trace
constexpr int RC_THREADS = 320;  // warp 2 TMA, warp 3 MMA, warps 0,1,8,9 row statistics, warps 4-7 epilogue

// store slots of the rows of kvd_checkpoint_residual_step (one new row per sequence of a batch)
struct CkptSlots {
  long long slot[KVD_MAX_STORE_RANGES];
};

constexpr int RC_MAX_JOBS = 65;  // row sources per launch: up to 64 store ranges and one caller buffer

// One source of rows inside a launch.  Jobs own consecutive runs of 256-row blocks.
struct RcJob {
  int mb_start;  // first 256-row block of this job in the launch
  int n;         // rows
  int row0;      // first row: index into the store slab, or 0 for a caller buffer
  int slab;      // store slab (sequence slot of this layer), or -1: rows come from the caller's buffer
  const int32_t *positions;  // [n]
  const float *sumsq;        // [n] sum of squares of each row (store ranges), nullptr for the caller's rows
  const float *scale;        // [n] FP8 store: the rows' quantisation scales; nullptr for bf16 rows
  __nv_bfloat16 *k_out;      // row m of the job at k_out + m * out_row_stride
  __nv_bfloat16 *v_out;
};

struct RecomputeParams {
  int n_jobs;
  int num_k_blocks;  // d_hidden / 64
  int num_m_blocks;  // over all jobs
  int num_n_blocks;
  int k_cols;  // n_kv * d_head: fused columns below this index are keys, the rest values
  long long out_row_stride;
  float inv_d_hidden;
  float rms_eps;
  int qk_norm;
  float qk_eps;
  int rope_style;
  const float2 *rope_hi;  // [n_hi][d_head/2] (cos, sin) of (pos & ~15) * freq_i
  const float2 *rope_lo;  // [d_head/2][16]   (cos, sin) of (pos & 15) * freq_i, pair-major
  int max_pos;            // positions must be in [0, max_pos)
  const float *gamma_k;   // [d_head] fp32 or nullptr
  int *status;
  unsigned long long timeout_ns;
  long long *trace;  // nullptr unless a trace buffer is attached
  const __nv_bfloat16 *ext_rows;  // the caller's rows (job with slab < 0), [n][d_hidden]
  int row_chunks;                 // d_hidden / 8: 16-byte chunks per row
  int wide_store;                 // outputs are 32-byte aligned: 32-byte stores
  const float *w_scale;           // FP8 variant: the weight matrix's quantisation scale (one float), else nullptr
  int store_rows;                 // rows per (layer, sequence) slab of the store (checking build)
  long long rows_out_stride;      // row stride of the caller rows' K/V outputs (the store ranges use out_row_stride)
  // STORE_RESIDUAL riding in the launch (kvd_decode_step_kv): caller row i is also written to slot append_slot[i]
  // of the store (rows, position, statistic), by the statistics warps that read it anyway
  int append_n;                   // 0: nothing is appended
  uint4 *append_rows;             // the store's rows, 16-byte chunks; slot s at append_rows + s * row_chunks
  int32_t *append_pos;
  float *append_sumsq;
  long long append_slot[RC_INLINE_STAT_ROWS];
  RcJob jobs[RC_MAX_JOBS];
};

// Fused recompute + attention (the recomputed K/V of a store range are consumed inside the kernel and
// never written): per job, the query of the range's sequence and where its partials go.
struct RcAttend {
  const __nv_bfloat16 *q;  // [n_q][d_head] of the job's sequence; nullptr: plain job, K and V are stored
  int q_pos;               // position of the query
  int lo_pos;              // first visible position (sliding window), 0 without a window
  int part_base;           // slot of the job's first 256-row block in the partial arrays
  int reserved;
};
struct FusedParams {
  float *part_o;   // [slot][n_q][d_head] unnormalised outputs
  float *part_ml;  // [slot][n_q][2] (max in log2 units, sum)
  int n_q;
  float scale_log2e;
  RcAttend att[RC_MAX_JOBS];
};
struct NoFusedParams {};

// ------------------------------------------------------------------------------ decode attention
constexpr int AT_THREADS = 128;        // streaming kernel
constexpr int AT_WARPS = 4;
constexpr int AT_CTAS_PER_SM = 4;      // 128 registers per thread
constexpr int AT_MERGE_THREADS = 640;  // merge kernel: at most 20 warps (102 registers each)
constexpr int AT_MERGE_WARPS = 20;
constexpr int AT_MERGE_SLICE = 64;     // channels per merge CTA
// partials one warp of the merge kernel fetches at once: 4*G registers each, 64 registers in all
constexpr int attn_merge_group(int g) { return 16 / g >= 1 ? 16 / g : 1; }
constexpr int AT_UNROLL = 8;          // keys per lane group per iteration
constexpr int AT_MAX_SEQS = 64;       // sequences per launch (bounded by the kernel parameter space)

struct AttnSeq {
  const __nv_bfloat16 *k[KVD_MAX_SEGMENTS];
  const __nv_bfloat16 *v[KVD_MAX_SEGMENTS];
  long long stride[KVD_MAX_SEGMENTS];
  int first[KVD_MAX_SEGMENTS];
  int len[KVD_MAX_SEGMENTS];
  int q_pos;
  int lo_pos;       // first visible position
  int hi_pos;       // last visible position (<= q_pos)
  int chunk0_pos;   // position of the first key of chunk 0 (multiple of the chunk size)
  int n_chunks;
  int part_base;    // chunks of the sequences before this one in the launch (the flattened grid)
  int iters;        // warp iterations per chunk
  int slot_base;    // slot of this sequence's chunk 0 in the partial arrays
  int merge_base;   // first slot and number of slots the merge kernel combines for this sequence: the
  int merge_count;  // streaming kernel's chunks, preceded by partials of the fused recompute kernel if any
};

// Launch-wide fields, followed by the per-sequence descriptors.  The kernel takes the variant whose
// array is just large enough (AttnLaunchT<4> for small batches: a 10 KB parameter block costs
// microseconds to launch).
struct AttnLaunchHead {
  int n_seqs;
  int total_chunks;
  int n_q;
  int n_kv;
  float scale_log2e;
  const __nv_bfloat16 *q;  // [n_seqs, n_q, d_head] (already offset to the launch's first sequence)
  __nv_bfloat16 *out;      // [n_seqs, n_q, d_head]
  float *part_o;           // [parts][n_q][d_head]
  float *part_ml;          // [parts][n_q][2]
  int *status;             // device status word (nullptr: none), used by the checking build
  int max_parts;           // slots the partial arrays hold
};
template <int NSEQ>
struct AttnLaunchT : AttnLaunchHead {
  AttnSeq seq[NSEQ];
};
typedef AttnLaunchT<AT_MAX_SEQS> AttnLaunch;

// keys per chunk for a head size and iteration count
inline int attn_keys_per_warp_iter(int d_head) { return (32 / (d_head / 8)) * AT_UNROLL; }
// Iterations per chunk.  Spans up to 8192 keys are cut into at most 128 chunks per (sequence, KV
// head), longer ones so that one sequence yields about 592 work units (chunks x KV heads) -- four
// CTAs on each of a B200's 148 SMs -- which keeps every SM equally loaded when the batch is 1.  A
// chunk is at least two iterations: a CTA's prologue and combine cost as much as streaming a few
// dozen keys, and in batched launches one-iteration CTAs measured 20 % slower.  A function of the
// model and of the visible span only, so a full cache and a recomputed + window + current layout
// of the same positions are split identically, and a sequence's result does not depend on what
// else is in the batch.
inline int attn_target_chunks(int n_kv, int span) {
  if (span <= 8192) return 128;
  const int t = (148 * AT_CTAS_PER_SM) / n_kv;
  return t > 16 ? t : 16;
}
inline int attn_iters_for_span(int d_head, int n_kv, int span) {
  const int per_iter = attn_keys_per_warp_iter(d_head) * AT_WARPS;
  const long long per_chunk_min = static_cast<long long>(per_iter) * attn_target_chunks(n_kv, span);
  long long iters = (span + per_chunk_min - 1) / per_chunk_min;
  if (iters < 2) iters = 2;
  if (iters > 64) iters = 64;
  return static_cast<int>(iters);
}
inline int attn_chunk_keys(int d_head, int iters) { return attn_keys_per_warp_iter(d_head) * AT_WARPS * iters; }
inline int attn_max_chunks(int d_head, int n_kv, int max_tokens) {
  const int per_iter = attn_keys_per_warp_iter(d_head) * AT_WARPS;
  const int capped = max_tokens / (per_iter * 64) + 2;  // once the iteration count is capped
  int target = attn_target_chunks(n_kv, max_tokens);
  if (target < 128) target = 128;
  return (capped > target ? capped : target) + 2;
}

// ------------------------------------------------------------------------------ context
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct RopeTable {
  float2 *hi = nullptr;
  float2 *lo = nullptr;
  int n_hi = 0;
};

struct LayerState {
  bool set = false;
  __nv_bfloat16 *wt = nullptr;  // [2*n_kv*d_head, d_hidden]: gamma-folded, K-major
  float *gamma_k = nullptr;     // [d_head] fp32
  float theta = 0.f;
  int window = 0;
  RopeTable rope;
  CUtensorMap tmap_b;
  // FP8 variant: E4M3 codes of W' / w_scale8, K-major; one scale for the matrix (device float)
  uint8_t *wt8 = nullptr;
  float *w_scale8 = nullptr;
  CUtensorMap tmap_b8;
};

}  // namespace kvd

struct kvd_ctx {
  kvd_model_desc desc;
  int device = 0;
  int num_sms = 0;
  int block_n = 0;
  int dtype = 0;  // 16-bit element type of rows, weights and K/V: 0 bf16, 1 fp16 (recompute path only)
  std::vector<kvd::LayerState> layers;
  std::map<uint32_t, kvd::RopeTable> rope_cache;  // keyed by the bits of theta
  // residual store
  __nv_bfloat16 *store_rows = nullptr;
  int32_t *store_pos = nullptr;
  float *store_sumsq = nullptr;
  float *ext_sumsq = nullptr;     // statistics of caller rows taken ahead of the recompute kernel
  size_t ext_sumsq_rows = 0;
  unsigned long long *argmax_keys = nullptr;  // scaffold greedy pick: one slot per row
  size_t argmax_rows = 0;
  int32_t *zero_pos = nullptr;    // ext_sumsq_rows zeros: the positions of rows that are not rotated (scaffold products)
  int layers_stored = 0;
  std::vector<int> rows_stored;  // [layers_stored * max_seqs]
  std::vector<CUtensorMap> store_maps;  // per stored layer: [max_seqs][max_tokens_per_seq][d_hidden]
  // FP8 residual store (separate arena): codes, positions, sums of squares of the original rows, scales
  uint8_t *store8_codes = nullptr;
  int32_t *store8_pos = nullptr;
  float *store8_sumsq = nullptr;
  float *store8_scale = nullptr;
  int layers_stored8 = 0;
  std::vector<int> rows_stored8;
  std::vector<CUtensorMap> store8_maps;
  // FP4 residual store (a third arena): E2M1 codes, E4M3 block scales, positions, sums of squares, row scales
  uint8_t *store4_codes = nullptr;
  uint8_t *store4_block = nullptr;
  int32_t *store4_pos = nullptr;
  float *store4_sumsq = nullptr;
  float *store4_scale = nullptr;
  int layers_stored4 = 0;
  std::vector<int> rows_stored4;
  unsigned *amax_scratch = nullptr;  // one word, used while weights are prepared
  // attention scratch
  float *part_o = nullptr;
  float *part_ml = nullptr;
  size_t workspace_bytes = 0;
  int max_parts = 0;
  int *d_status = nullptr;
  uint64_t launches = 0;
  uint64_t prepared_bytes = 0;
  unsigned long long timeout_ns = 2000000000ull;
  long long *trace = nullptr;
  size_t trace_bytes = 0;
  std::string last_error;
  kvd::EncodeTiledFn encode = nullptr;
};

namespace kvd {
// Kernels are launched as programmatic dependents of their predecessor in the stream unless the
// environment variable KVD_SERIAL_LAUNCH says otherwise: a bit mask, 1 = recompute kernel, 2 = attention
// streaming kernel, 4 = attention merge kernel get plain stream ordering instead.
inline int serial_launch_mask() {
  static const int mask = [] {
    const char *e = getenv("KVD_SERIAL_LAUNCH");
    return e ? atoi(e) : 0;
  }();
  return mask;
}

// launchers implemented next to their kernels
kvd_status launch_recompute(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                            const CUtensorMap &tmap_rows, const RecomputeParams &p, cudaStream_t stream);
kvd_status launch_recompute_fused(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                                  const CUtensorMap &tmap_rows, const RecomputeParams &p, const FusedParams &fp,
                                  cudaStream_t stream, int eb = 2);
kvd_status launch_attention(kvd_ctx *ctx, const AttnLaunch &L, int d_head, int group, cudaStream_t stream);
kvd_status launch_prepare_weights(kvd_ctx *ctx, const __nv_bfloat16 *w, const __nv_bfloat16 *gamma, __nv_bfloat16 *wt,
                                  int d_hidden, int n_cols, cudaStream_t stream);
kvd_status launch_convert_gamma(kvd_ctx *ctx, const __nv_bfloat16 *g, float *out, int n, cudaStream_t stream);
kvd_status launch_rowstats(kvd_ctx *ctx, const __nv_bfloat16 *rows, float *sumsq, int n, int d_hidden,
                           cudaStream_t stream);
kvd_status launch_checkpoint_fp8(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, uint8_t *dst_codes,
                                 int32_t *dst_pos, float *dst_sumsq, float *dst_scale, int n, int d_hidden,
                                 cudaStream_t stream);
kvd_status launch_prepare_weights_fp8(kvd_ctx *ctx, const __nv_bfloat16 *w, const __nv_bfloat16 *gamma, uint8_t *wt8,
                                      int d_hidden, int n_cols, unsigned *amax_scratch, float *scale_out,
                                      cudaStream_t stream);
kvd_status launch_recompute_fp8(kvd_ctx *ctx, const LayerState &ls, const CUtensorMap &tmap_store,
                                const CUtensorMap &tmap_rows, const RecomputeParams &p, cudaStream_t stream);
kvd_status launch_checkpoint(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, __nv_bfloat16 *dst_rows,
                             int32_t *dst_pos, float *dst_sumsq, int n, int d_hidden, cudaStream_t stream);
kvd_status launch_selftest_bounds(kvd_ctx *ctx, cudaStream_t stream);
kvd_status launch_checkpoint_scatter(kvd_ctx *ctx, const __nv_bfloat16 *rows, const int32_t *pos, const CkptSlots &slots,
                                     int n, int d_hidden, cudaStream_t stream);
// kvd_prefill_attention: many query tokens of one sequence, tiled over query rows (Eq. 6-7 per row)
struct PrefillParams {
  const __nv_bfloat16 *q;    // [n_rows][n_q][d_head]
  __nv_bfloat16 *out;        // [n_rows][n_q][d_head]
  const int32_t *q_pos;      // DEVICE [n_rows]
  int n_rows, n_q, n_kv, window;
  float scale_log2e;
  int seg_lo, seg_hi;        // first and last position any segment holds
  const __nv_bfloat16 *k[KVD_MAX_SEGMENTS];
  const __nv_bfloat16 *v[KVD_MAX_SEGMENTS];
  long long stride[KVD_MAX_SEGMENTS];
  int first[KVD_MAX_SEGMENTS];
  int len[KVD_MAX_SEGMENTS];
  int *status;                    // device status word
  unsigned long long timeout_ns;  // limit of every in-kernel wait
};
// the tcgen05 form of the call (128 MMA rows per CTA, scores and outputs in tensor memory)
kvd_status launch_prefill_tc(kvd_ctx *ctx, const PrefillParams &P, int d_head, int group, cudaStream_t stream);
kvd_status launch_selftest_timeout(kvd_ctx *ctx, unsigned long long timeout_ns, cudaStream_t stream);
kvd_status cuda_fail(kvd_ctx *ctx, cudaError_t e, const char *where);
// host helpers shared by the entry points (kvd_api.cu)
kvd_status encode_2d(kvd_ctx *ctx, CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer,
                     uint32_t box_inner, uint32_t box_outer, int eb = 2);
kvd_status encode_rows_3d(kvd_ctx *ctx, CUtensorMap *map, const void *base, uint64_t d_hidden, uint64_t rows,
                          uint64_t slabs, int eb = 2);
kvd_status get_rope(kvd_ctx *ctx, float theta, RopeTable *out);
}  // namespace kvd
