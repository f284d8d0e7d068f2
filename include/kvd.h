/*
 * kvd.h -- C ABI of the KV-Direct hot path for NVIDIA B200 (sm_100a).
 *
 * KV-Direct keeps, for every token, the residual row that entered each decoder layer instead of
 * the layer's key/value pair, and rebuilds keys and values when attention needs them
 * (paper Section 3.4, Algorithm 1; reconstruction identities Eq. 13-14).  This library is the
 * per-layer hot path of that scheme:
 *
 *   kvd_checkpoint_residual  STORE_RESIDUAL(C, l) of Algorithm 1: append residual rows to the store.
 *   kvd_recompute_kv         RECOMPUTE_KV(C, l): RMSNorm (Eq. 1-2) -> fused [W_K | W_V] projection
 *                            (Eq. 13-14) -> optional per-head key norm -> rotation of the keys at each
 *                            row's stored position (Eq. 11-12).  The same call produces the current
 *                            token's (K_t, V_t), so "first pass" and "recomputed" K/V are the output
 *                            of one routine and are bit-identical for the same row and position.
 *   kvd_recompute_kv_step    the K/V work of one decode step of a layer in one launch: RECOMPUTE_KV
 *                            for the evicted ranges of every sequence plus (K_t, V_t) of the new tokens.
 *   kvd_decode_attention     ATTENTION(Q, K_all, V_all) for one query token per sequence (Eq. 6-7)
 *                            over the CONCAT of up to four position-contiguous K/V segments
 *                            (recomputed, live window, current token), grouped-query heads,
 *                            optional sliding-window mask.
 *
 * General rules
 *   - Plain C.  Every pointer documented as DEVICE points to memory on the context's GPU that the
 *     caller allocated and keeps alive until the work enqueued on `stream` has finished; the
 *     library never frees or reallocates it.  HOST pointers are read before the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All kernels
 *     are enqueued asynchronously on it; no call synchronises the device except kvd_create,
 *     kvd_set_layer (one-time preparation), kvd_poll_status and kvd_destroy.
 *   - Every call returns a kvd_status and never throws, aborts or traps the device.  Argument
 *     errors are detected on the host before anything is launched.  Conditions that only the
 *     device can see (a position outside [0, max_tokens_per_seq), a pipeline wait that ran out)
 *     are recorded in a device status word that kvd_poll_status reads.
 *   - bf16 everywhere a tensor is stored; fp32 accumulation and fp32 epilogue arithmetic.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x kvd_create fails.
 *   - Kernels after the first of a call sequence are launched as programmatic dependents of their
 *     predecessor in the stream (their set-up overlaps its tail; they wait for its completion before
 *     touching its results), which is transparent to callers and to stream capture.  Environment:
 *     KVD_SERIAL_LAUNCH (bit mask: 1 recompute, 2 attention streaming, 4 attention merge) restores
 *     plain stream ordering for those kernels; KVD_SPIN_LIMIT_MS (read by kvd_create) bounds every
 *     in-kernel pipeline wait (default 2000 ms).
 */
#ifndef KVD_H_
#define KVD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvd_ctx kvd_ctx; /* opaque; one per model per device */

typedef enum {
  KVD_OK = 0,
  KVD_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, index out of range            */
  KVD_ERR_SHAPE = 2,       /* dimensions the kernels do not cover                          */
  KVD_ERR_ALIGNMENT = 3,   /* a pointer or stride is not 16-byte aligned                   */
  KVD_ERR_CAPACITY = 4,    /* store, workspace or batch limit exceeded                     */
  KVD_ERR_STATE = 5,       /* call made before its prerequisite (layer not set, ...)       */
  KVD_ERR_UNSUPPORTED = 6, /* no usable device / driver entry point                        */
  KVD_ERR_CUDA = 7,        /* a CUDA runtime call failed; see kvd_last_cuda_error          */
  KVD_ERR_TIMEOUT = 8,     /* a bounded wait inside a kernel expired (from kvd_poll_status) */
  KVD_ERR_POSITION = 9,    /* a row's position was outside [0, max_tokens_per_seq)         */
  KVD_ERR_BOUNDS = 10      /* checking build only: a kernel met an index outside its table or buffer */
} kvd_status;

/* Pairing of channels rotated together by Eq. 11-12. */
typedef enum {
  KVD_ROPE_INTERLEAVED = 0, /* (2i, 2i+1): the pairing Eq. 11-12 print            */
  KVD_ROPE_HALF = 1         /* (i, i + d_head/2): the same rotation after a fixed
                               channel permutation of q and k                      */
} kvd_rope_style;

/* Model-wide constants.  Supported: d_hidden % 64 == 0; d_head in {64, 128, 256};
 * n_q_heads % n_kv_heads == 0 with a group size of 1..8; 2*n_kv_heads*d_head % 128 == 0. */
typedef struct {
  int32_t n_layers;
  int32_t d_hidden;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t d_head;
  float rms_eps;              /* added to mean(x^2) inside the root of Eq. 2 (the paper prints none) */
  int32_t qk_norm;            /* 1: RMS-normalise every key head over d_head before the rotation      */
  float qk_norm_eps;
  int32_t rope_style;         /* kvd_rope_style                                                         */
  int32_t max_seqs;           /* sequences the residual store can hold                                  */
  int32_t max_tokens_per_seq; /* rows per (layer, sequence) in the store; also the position bound       */
  int32_t max_batch;          /* largest `batch` of kvd_decode_attention (sizes the workspace)          */
} kvd_model_desc;

/* One layer's frozen parameters (all DEVICE, bf16, read during kvd_set_layer only). */
typedef struct {
  const void *w_kv;       /* [d_hidden, 2*n_kv*d_head] row-major: W_K columns (head-major) then W_V columns */
  const void *gamma_in;   /* [d_hidden] effective RMSNorm scale gamma of Eq. 1                               */
  const void *gamma_k;    /* [d_head] key-norm scale shared by all heads; NULL when qk_norm == 0             */
  float rope_theta;       /* base b of Eq. 11-12                                                             */
  int32_t sliding_window; /* 0: global layer.  w > 0: a key is visible iff 0 <= q_pos - key_pos < w          */
} kvd_layer_desc;

/* A run of keys/values at consecutive positions first_pos .. first_pos+len-1 (DEVICE, bf16).
 * Element (j, h, c) of k is at k[j*row_stride + h*d_head + c]; likewise v.  row_stride is in
 * elements and a multiple of 8; k and v are 16-byte aligned.  Segments of one sequence must not
 * overlap in position. */
typedef struct {
  const void *k;
  const void *v;
  int64_t row_stride;
  int32_t first_pos;
  int32_t len;
} kvd_kv_segment;

#define KVD_MAX_SEGMENTS 4

/* Byte counts reported by kvd_memory_stats.  The eq* fields are the paper's closed forms for the
 * numbers of tokens currently stored; the others are what this context actually occupies. */
typedef struct {
  uint64_t checkpoint_bytes_used;     /* rows + positions + statistics currently held (all stores)       */
  uint64_t checkpoint_bytes_capacity; /* size the attached arenas must have (all stores)                  */
  uint64_t workspace_bytes;           /* attention scratch (split partials)                               */
  uint64_t prepared_weight_bytes;     /* gamma-folded K-major copies of W_kv, rotation tables, key scales */
  uint64_t tokens_stored;             /* max over layers of the rows stored, summed over sequences        */
  uint64_t eq23_kv_bytes_per_token;   /* 2 L n_kv d_head b                                                */
  uint64_t eq24_residual_bytes_per_token; /* d_hidden b (one vector per token, the paper's accounting)    */
  uint64_t per_layer_residual_bytes_per_token; /* L d_hidden b (what per-layer recomputation stores)      */
} kvd_mem_stats;

/* Create a context on the current CUDA device.  HOST desc.  Fails with KVD_ERR_UNSUPPORTED when the
 * device is not compute capability 10.x, KVD_ERR_SHAPE for dimensions outside the supported set. */
kvd_status kvd_create(const kvd_model_desc *desc, kvd_ctx **out);

/* Release everything the context allocated (prepared weights, tables).  Synchronises the device. */
void kvd_destroy(kvd_ctx *ctx);

/* Element type of residual rows, weights, K/V, queries and attention outputs.  bf16 is the default and the
 * only type the FP8 and static entry points accept (KVD_ERR_UNSUPPORTED otherwise); fp16 exists for
 * kvd_checkpoint_residual / kvd_recompute_kv / kvd_recompute_kv_step / kvd_decode_step_kv / kvd_decode_attention /
 * kvd_decode_attention_rows / kvd_decode_attention_recompute, fp32 for the checkpoint and recompute calls (rows, weights and K/V outputs are fp32, strides count fp32 elements, the tensor cores read the
 * operands as TF32 and accumulate in fp32) -- the reconstruction identities (Eq. 13-14) do not depend on the
 * element type, and the bitwise recompute-equals-first-pass check of the paper's Section 5.1 is run in all
 * three.  Call before kvd_set_layer, kvd_attach_store (when the element size changes) and any checkpoint
 * (KVD_ERR_STATE after). */
#define KVD_DTYPE_BF16 0
#define KVD_DTYPE_F16 1
#define KVD_DTYPE_F32 2
kvd_status kvd_set_dtype(kvd_ctx *ctx, int dtype);
/* kvd_store_bytes for a context of the given element type (fp32 rows take twice the room). */
size_t kvd_store_bytes_dtype(const kvd_model_desc *desc, int layers_stored, int dtype);

/* Prepare layer `layer`: build W' = diag(gamma_in) * W_kv rounded to the context's element type and stored K-major, the
 * fp32 key-norm scale, and the rotation tables for rope_theta.  Folding gamma into W is Eq. 1
 * composed with Eq. 13-14: (x / rms * gamma) W = (x W') / rms.  Enqueues on `stream` and waits for it. */
kvd_status kvd_set_layer(kvd_ctx *ctx, int layer, const kvd_layer_desc *ldesc, void *stream);

/* Bytes the residual store needs for `layers_stored` layers (rows + positions + row statistics). */
size_t kvd_store_bytes(const kvd_model_desc *desc, int layers_stored);

/* Hand the context a caller-owned DEVICE arena (256-byte aligned, >= kvd_store_bytes) for the
 * residual store C of Algorithm 1.  Resets all row counts to zero.
 * Layout (the arena stays the caller's, who may read it): residual rows as bf16
 * [layers_stored][max_seqs][max_tokens_per_seq][d_hidden] from the start of the arena, then, at the
 * next multiple of 256 bytes, their positions as int32 [layers_stored][max_seqs][max_tokens_per_seq],
 * then, again at the next multiple of 256 bytes, the sum of squares of each row as fp32 in the same
 * shape (the RMSNorm statistic of Eq. 2, taken once when the row is checkpointed and read back by every
 * recomputation; a caller that writes rows into the arena itself must write these too).
 * Row r of (layer, seq) is valid for r < kvd_rows_stored(ctx, layer, seq). */
kvd_status kvd_attach_store(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored);

/* Forget the rows of one sequence (all layers) so that its slot can be reused. */
kvd_status kvd_reset_sequence(kvd_ctx *ctx, int seq);

/* Rows currently stored for (layer, seq); negative on bad arguments. */
int kvd_rows_stored(const kvd_ctx *ctx, int layer, int seq);

/* Bytes of attention scratch for the context's max_batch / max_tokens_per_seq. */
size_t kvd_workspace_bytes(const kvd_model_desc *desc);

/* How decode attention splits one sequence: the keys at positions first_visible .. last_visible (after
 * the window and the query position have been applied) are cut into chunks aligned to multiples of
 * *chunk_keys; returns the number of chunks (= partials per KV head that the call keeps in its scratch)
 * and, if not NULL, stores the chunk length.  A function of its arguments only: the split of a sequence
 * does not depend on the segment layout or on the rest of the batch.  Host-only; 0 on bad arguments
 * (d_head not in {64, 128, 256}, n_kv_heads < 1, an empty or negative range). */
int kvd_attention_split(int d_head, int n_kv_heads, int first_visible, int last_visible, int *chunk_keys);

/* Hand the context a caller-owned DEVICE workspace (256-byte aligned, >= kvd_workspace_bytes). */
kvd_status kvd_attach_workspace(kvd_ctx *ctx, void *workspace, size_t bytes);

/* STORE_RESIDUAL(C, l): append n residual rows (DEVICE bf16 [n, d_hidden], 16-byte aligned) and
 * their absolute positions (DEVICE int32 [n]) to the store of (layer, seq), together with each row's
 * sum of squares (taken in the one fixed order that recomputation from caller rows uses as well).
 * KVD_ERR_CAPACITY when the rows do not fit; KVD_ERR_STATE without an attached store. */
kvd_status kvd_checkpoint_residual(kvd_ctx *ctx, int seq, int layer, const void *rows, const int32_t *positions,
                                   int n, void *stream);

/* STORE_RESIDUAL(C, l) for one decode step of a batch, in ONE launch: row i of rows (DEVICE bf16
 * [n, d_hidden], 16-byte aligned; positions DEVICE int32 [n]) is appended to the store of (layer, seqs[i]),
 * exactly as kvd_checkpoint_residual would append it (same bits, same statistic).  seqs is a HOST array of
 * n <= KVD_MAX_STORE_RANGES sequence slots; a slot may occur more than once (its rows are appended in order).
 * Nothing is stored when any entry is rejected. */
kvd_status kvd_checkpoint_residual_step(kvd_ctx *ctx, int layer, int n, const int32_t *seqs, const void *rows,
                                        const int32_t *positions, void *stream);

/* RECOMPUTE_KV(C, l), Eq. 13-14.
 *   rows != NULL: DEVICE bf16 [n, d_hidden] (16-byte aligned) with DEVICE int32 positions[n];
 *                 seq and first_row are ignored.  This is also how (K_t, V_t) of new tokens is made.
 *   rows == NULL: rows first_row .. first_row+n-1 of the store of (layer, seq) with their stored
 *                 positions; `positions` must be NULL.
 *   k_out, v_out: DEVICE bf16; row m, head h, channel c at [m*out_row_stride + h*d_head + c]
 *                 (out_row_stride in elements, multiple of 8, >= n_kv*d_head; bases 16-byte aligned).
 * n == 0 is a no-op.  Output bits for a row depend only on that row, its position and the layer,
 * never on n, on the row's index in the batch, or on whether the row came from the store or from the
 * caller.  Rows from the store use the statistic stored with them; for more than 64 caller rows the call
 * first launches a small kernel that takes their statistics into a scratch of the context (calls on one
 * context are stream-ordered by contract: they must not overlap on different streams).  Outputs whose
 * bases are 32-byte aligned and whose row stride is a multiple of 16 elements are written with 32-byte
 * stores (a little faster); 16-byte alignment is all that is required. */
kvd_status kvd_recompute_kv(kvd_ctx *ctx, int layer, const void *rows, const int32_t *positions, int n, int seq,
                            int first_row, void *k_out, void *v_out, int64_t out_row_stride, void *stream);

/* One range of checkpointed rows of one sequence, for kvd_recompute_kv_step. */
typedef struct kvd_store_range {
  int32_t seq;       /* sequence slot */
  int32_t first_row; /* first stored row of (layer, seq) */
  int32_t n;         /* rows; 0 = skip this entry */
  int32_t reserved;  /* 0 */
  void *k_out;       /* DEVICE bf16, row m of the range at [m*out_row_stride + h*d_head + c] */
  void *v_out;
} kvd_store_range;
#define KVD_MAX_STORE_RANGES 64

/* The K/V work of one decode step of one layer in ONE launch (Algorithm 1, inside the layer loop):
 * RECOMPUTE_KV(C, l) for the evicted tokens of every sequence of the batch (Eq. 13-14) together
 * with the projection that makes (K_t, V_t) of the new tokens.  Equivalent to one kvd_recompute_kv
 * call per range plus one for `rows`, with identical output bits; the rows of all sources share
 * the kernel's tile schedule, so single-token sources cost no launch of their own.
 *   ranges    HOST array of n_ranges <= KVD_MAX_STORE_RANGES entries (read during the call only).
 *   rows      DEVICE bf16 [n_rows, d_hidden] (16-byte aligned) with DEVICE int32 positions[n_rows],
 *             results to k_rows_out / v_rows_out; n_rows == 0 leaves this source out.
 *   out_row_stride applies to every output (elements, multiple of 8, >= n_kv*d_head).
 * Errors as kvd_recompute_kv; nothing is launched when any entry is rejected. */
kvd_status kvd_recompute_kv_step(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                 const void *rows, const int32_t *positions, int n_rows, void *k_rows_out,
                                 void *v_rows_out, int64_t out_row_stride, void *stream);

/* Everything a decode step of one layer does to K/V and to the store, in ONE launch (Algorithm 1, inside the
 * layer loop): STORE_RESIDUAL(C, l) for the new tokens, RECOMPUTE_KV(C, l) for the evicted ranges (Eq. 13-14) and
 * (K_t, V_t) of the new tokens.  As kvd_recompute_kv_step, with two additions:
 *   append_seqs  HOST int32 [n_rows] or NULL.  Not NULL: row i of `rows` is also appended to the store of
 *                (layer, append_seqs[i]) -- rows, position and sum of squares, the same bits
 *                kvd_checkpoint_residual would store -- by the warps of the kernel that read the rows for
 *                their statistics anyway; n_rows <= 64 (KVD_ERR_CAPACITY beyond).  The appended rows are not
 *                visible to `ranges` of the same call.
 *   rows_out_row_stride  row stride (elements, multiple of 8, >= n_kv*d_head; <= 0 selects n_kv*d_head) of
 *                k_rows_out / v_rows_out alone, so that the new tokens' K and V can be written straight into
 *                a cache laid out [sequence][position][n_kv*d_head] (stride = positions per sequence x
 *                n_kv*d_head, base = the slot of the current position) while the recomputed ranges go to a
 *                scratch with out_row_stride.
 * Output bits are those of the separate calls.  Nothing is launched or stored when any argument is rejected. */
kvd_status kvd_decode_step_kv(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                              int64_t out_row_stride, const void *rows, const int32_t *positions, int n_rows,
                              const int32_t *append_seqs, void *k_rows_out, void *v_rows_out,
                              int64_t rows_out_row_stride, void *stream);

/* ---- FP8 checkpoints (lower-precision residual rows and weights: the second future-work item of the
 * paper's Section 6, which fixes no format; this is the definition this library implements) ----
 * A residual row x (bf16) is stored as E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits,
 * largest finite value 448) with one fp32 scale per row:
 *     s_x = max|x| / 448,    code_k = e4m3(x_k * (448 / max|x|))   round to nearest even, saturating, all in fp32,
 * together with its position and the sum of squares of the ORIGINAL row (1/rms of Eq. 2 is not affected by
 * the quantisation).  The folded weights W' = gamma (.) W_kv get one scale for the whole matrix,
 * s_w = max|W'| / 448, code = e4m3(W' * (448 / max|W'|)) (prepared by kvd_set_layer next to the bf16 copy).
 * RECOMPUTE_KV from such rows is Eq. 13-14 on the dequantised operands,
 *     y = (s_x s_w / rms(x)) * sum_k code_x[k] code_w[k][:],   then key norm and rotation as usual,
 * with the code products accumulated on the tensor cores (kind f8f6f4, fp32 accumulation).  Per token and
 * layer the store holds d_hidden + 12 bytes instead of 2 d_hidden + 8.  The result is NOT the bf16 result:
 * each operand carries up to 2^-4 relative error, a few per cent of the outputs' rms after the contraction
 * (measured in the tests); exactness claims (Prop. 3.2) do not carry over, determinism does (a row's bits
 * do not depend on the batch it is recomputed in).
 * The FP8 store is a second, independent arena (layout: codes uint8 [layers][max_seqs][max_tokens][d_hidden],
 * then positions int32, sums of squares fp32, scales fp32, each [layers][max_seqs][max_tokens] and each
 * region starting at a 256-byte multiple) with row counts of its own (kvd_reset_sequence_fp8).
 * kvd_store_bytes_fp8 returns 0 for shapes the variant does not support (d_hidden % 16 != 0). */
size_t kvd_store_bytes_fp8(const kvd_model_desc *desc, int layers_stored);
kvd_status kvd_attach_store_fp8(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored);
int kvd_rows_stored_fp8(const kvd_ctx *ctx, int layer, int seq);
kvd_status kvd_reset_sequence_fp8(kvd_ctx *ctx, int seq);
/* Append n rows (DEVICE bf16 [n, d_hidden], 16-byte aligned; DEVICE int32 positions[n]) in quantised form. */
kvd_status kvd_checkpoint_residual_fp8(kvd_ctx *ctx, int seq, int layer, const void *rows, const int32_t *positions,
                                       int n, void *stream);
/* RECOMPUTE_KV for ranges of the FP8 store (as kvd_recompute_kv_step without caller rows): K and V (bf16) of
 * rows first_row .. first_row+n-1 of every range to its k_out / v_out. */
kvd_status kvd_recompute_kv_fp8(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                int64_t out_row_stride, void *stream);
/* Rows in the FP8 checkpoint format that live in the caller's memory instead of the store (the new tokens of a
 * decode step: one contiguous buffer for the whole batch instead of one store range per sequence):
 * kvd_quantize_rows_fp8 turns n bf16 rows (DEVICE [n, d_hidden], 16-byte aligned) into codes (DEVICE uint8
 * [n, d_hidden], 16-byte aligned), scales and sums of squares (DEVICE fp32 [n]) exactly as
 * kvd_checkpoint_residual_fp8 would store them; a kvd_fp8_rows (HOST struct of DEVICE pointers; positions int32
 * [n]; k_out / v_out bf16 [n, out_row_stride], 16-byte aligned) hands them to the _rows forms of the FP8
 * recompute calls, which write their K and V like those of a store range (same bits as from the store).
 * rows == NULL or n == 0: no caller rows. */
typedef struct {
  const void *codes;
  const float *scales;
  const float *sumsq;
  const int32_t *positions;
  int32_t n;
  int32_t reserved;
  void *k_out;
  void *v_out;
} kvd_fp8_rows;
kvd_status kvd_quantize_rows_fp8(kvd_ctx *ctx, const void *rows, int n, void *codes_out, float *scales_out,
                                 float *sumsq_out, void *stream);
kvd_status kvd_recompute_kv_fp8_rows(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                     const kvd_fp8_rows *rows, int64_t out_row_stride, void *stream);

/* ---- FP4 checkpoints (the same future-work item; again the format is this library's definition) ----
 * A residual row x (bf16) is stored in 4 bits per channel with two levels of scales (the layout known as NVFP4,
 * the outer scale taken per row and restricted to a power of two):
 *     s_row = 2^(floor(log2 max|x|) - 10)                      (1 for an all-zero row; max|x| / s_row in [1024, 2048))
 *     b     = e4m3((max|x_block| / 6) / s_row)                 per block of 16 consecutive channels, fp32, nearest even
 *     c_k   = e2m1(x_k / (b * s_row))                          nearest of {0, .5, 1, 1.5, 2, 3, 4, 6}, ties to the even
 *                                                              code, saturating; all codes 0 when b rounds to 0
 * together with its position and the sum of squares of the ORIGINAL row.  A value decodes as c_k * b * s_row, which
 * is exact in bf16.  RECOMPUTE_KV from such rows is Eq. 13-14 on the decoded rows with 1/rms of the original row:
 * kvd_recompute_kv_fp4 expands the rows of its ranges into a caller-provided scratch (bf16 rows, positions,
 * statistics; kvd_fp4_scratch_bytes for the total row count of a call) and runs the ordinary bf16 projection on
 * them -- storage is 4-bit, the arithmetic is the bf16 path's; two launches.  Per token and layer the store holds
 * d_hidden/2 + d_hidden/16 + 12 bytes (1,452 for d_hidden = 2560; bf16 rows 5,128; the K/V they replace 4,096).
 * Accuracy is that of the format, reported by the tests, not claimed; exactness (Prop. 3.2) does not carry over,
 * determinism does.  The FP4 store is a third, independent arena: codes uint8 [layers][max_seqs][max_tokens]
 * [d_hidden/2] (channel 2j in the low nibble of byte j), block scales uint8 [...][d_hidden/16], positions int32,
 * sums of squares fp32, row scales fp32, each region starting at a 256-byte multiple.  d_hidden % 64 == 0 and
 * d_hidden <= 2560; bf16 contexts only. */
size_t kvd_store_bytes_fp4(const kvd_model_desc *desc, int layers_stored);
kvd_status kvd_attach_store_fp4(kvd_ctx *ctx, void *arena, size_t bytes, int layers_stored);
int kvd_rows_stored_fp4(const kvd_ctx *ctx, int layer, int seq);
kvd_status kvd_reset_sequence_fp4(kvd_ctx *ctx, int seq);
kvd_status kvd_checkpoint_residual_fp4(kvd_ctx *ctx, int seq, int layer, const void *rows, const int32_t *positions,
                                       int n, void *stream);
size_t kvd_fp4_scratch_bytes(const kvd_model_desc *desc, int max_rows);
/* ranges: rows first_row .. first_row+n-1 of the FP4 store of (layer, ranges[i].seq), K and V (bf16) to k_out / v_out
 * with row stride out_row_stride.  scratch: DEVICE, 256-byte aligned, >= kvd_fp4_scratch_bytes(desc, sum of n). */
kvd_status kvd_recompute_kv_fp4(kvd_ctx *ctx, int layer, const kvd_store_range *ranges, int n_ranges,
                                int64_t out_row_stride, void *scratch, size_t scratch_bytes, void *stream);

/* ATTENTION(Q, K_all, V_all) of Algorithm 1 for one new token per sequence (Eq. 6-7).
 *   q      DEVICE bf16 [batch, n_q_heads, d_head], already normalised and rotated to q_pos.
 *   q_pos  HOST int32 [batch]: position of each sequence's query token.
 *   segs   HOST [batch][n_segs] (n_segs <= KVD_MAX_SEGMENTS); len == 0 entries are skipped.
 *   scale  multiplies q.k before the softmax; <= 0 selects 1/sqrt(d_head) (Eq. 6).
 *   out    DEVICE bf16 [batch, n_q_heads, d_head].
 * Key j of a sequence is attended iff key_pos <= q_pos and, on a sliding-window layer,
 * q_pos - key_pos < window.  Query head h reads KV head h / (n_q_heads / n_kv_heads).  A sequence
 * with no visible key yields zeros.  The split of the keys into work units and the order in which
 * partial results are merged depend on key positions only, not on which segment holds a key, so a
 * full cache in one segment and the same keys spread over several segments give identical bits.
 * Needs an attached workspace. */
kvd_status kvd_decode_attention(kvd_ctx *ctx, int layer, int batch, const void *q, const int32_t *q_pos,
                                const kvd_kv_segment *segs, int n_segs, float scale, void *out, void *stream);

/* ATTENTION of Algorithm 1 for SEVERAL tokens of ONE sequence, each with its own causal limit (a prefill segment, or
 * the replay of an evicted prefix when only one residual row per token is kept): row i of q (DEVICE [n_rows,
 * n_q_heads, d_head]) is the query of the token at position q_pos[i] (HOST int32 [n_rows]) and attends the keys of
 * `segs` (HOST [n_segs]: the one sequence's segments, shared by all rows) at positions <= q_pos[i], inside the
 * layer's window.  out DEVICE [n_rows, n_q_heads, d_head].  Every row's result has the bits kvd_decode_attention
 * gives for that query alone: the rows go through the same kernels, as many per launch as the workspace's
 * partial slots hold (at most 64), so the call is a host loop over launches, not one launch. */
kvd_status kvd_decode_attention_rows(kvd_ctx *ctx, int layer, int n_rows, const void *q, const int32_t *q_pos,
                                     const kvd_kv_segment *segs, int n_segs, float scale, void *out, void *stream);

/* ATTENTION of Algorithm 1 (Eq. 6-7) for many tokens of one sequence in ONE launch, tiled over query rows on the
 * tensor cores: the prefill-shaped call.  Arguments as kvd_decode_attention_rows, except that q_pos is a DEVICE
 * int32 [n_rows] (nothing on the host depends on the positions).  Keys are taken in blocks of 64 aligned to absolute
 * position; the softmax weights are rounded to the element type before the second product (fp32 accumulation); a
 * row's weights are taken against a reference that follows its maximum in steps (it moves when a block exceeds it by
 * 2^8), which changes rounding, not the softmax.  Both products run as tcgen05.mma with scores and output in tensor
 * memory (CTA pairs at d_head 256); KVD_ERR_TIMEOUT from kvd_poll_status if an in-kernel wait ran out.
 * A row's result depends on that row, its position and the keys alone -- not on n_rows, on the row's index or on the
 * other rows of the call -- so a token attended alone and the same token inside a long call give the same bits.
 * They are NOT the bits of kvd_decode_attention / kvd_decode_attention_rows (another split of the keys): same
 * tolerance against the definition; use one of the two families throughout where outputs must be bit-identical.
 * bf16 and fp16 contexts; needs no workspace. */
kvd_status kvd_prefill_attention(kvd_ctx *ctx, int layer, int n_rows, const void *q, const int32_t *q_pos,
                                 const kvd_kv_segment *segs, int n_segs, float scale, void *out, void *stream);

/* RECOMPUTE_KV and ATTENTION of Algorithm 1 in one pass for the evicted tokens (Eq. 13-14 feeding
 * Eq. 6-7): the keys and values rebuilt from the residual rows of ranges[b] are consumed inside the
 * recompute kernel -- the rotated key of a row is multiplied with the queries of its KV head, the value
 * tile is produced transposed and summed over rows with the softmax weights -- and never written to
 * memory.  The result for sequence b is attention over [keys recomputed from ranges[b]] united with the
 * live segments segs[b][*] (window, current token), as kvd_recompute_kv_step followed by
 * kvd_decode_attention would give it, up to rounding: the recomputed part is split by 256-row blocks
 * instead of position chunks and its values are not rounded to bf16 on the way, so the bits differ from
 * the two-call path (same tolerances against the definition).  Use the two-call path where bit-identical
 * outputs across cache policies are required.
 *   ranges  HOST [batch]: rows first_row .. first_row+n-1 of the store of (layer, ranges[b].seq); k_out and
 *           v_out are ignored; n == 0 leaves a sequence with its live segments only.  Visibility of a
 *           recomputed key follows its stored position (<= q_pos[b], inside the layer's window).
 *   rows, positions, n_rows, k_rows_out, v_rows_out, out_row_stride: the new tokens, exactly as in
 *           kvd_recompute_kv_step -- their K and V ARE written (the live segments usually point at them).
 *   q, q_pos, segs, n_segs, scale, out: as in kvd_decode_attention; batch <= KVD_MAX_STORE_RANGES.
 *   The current token can be folded into the recomputed part: its row is checkpointed like every token's, so
 *   ranges[b] may end with it (n counts it) while `rows` still makes its K_t, V_t for a window that keeps them;
 *   when no live segment is left (n_segs == 0 or all lengths 0) the live-segment launch is skipped.
 * Three launches (recompute+attend, live segments, merge), two without live segments.  The fused form pays
 * where the recompute volume is large (kvd_fused_recompute_pays); below that the two-call sequence
 * kvd_recompute_kv_step + kvd_decode_attention is faster, because a unit of work here is a key tile AND a
 * value tile on one SM pair, where the plain kernel gives every tile its own.  KVD_ERR_UNSUPPORTED, with nothing launched,
 * for shapes the fused kernel is not built for (it exists for 256-column tiles with d_head 256 and 1 or 2
 * query heads per KV head, or d_head 128 and 1, 2 or 4); needs the store and the workspace attached. */
kvd_status kvd_decode_attention_recompute(kvd_ctx *ctx, int layer, int batch, const void *q, const int32_t *q_pos,
                                          const kvd_store_range *ranges, const void *rows,
                                          const int32_t *positions, int n_rows, void *k_rows_out, void *v_rows_out,
                                          int64_t out_row_stride, const kvd_kv_segment *segs, int n_segs,
                                          float scale, void *out, void *stream);

/* Host-only: 1 when the fused call (kvd_decode_attention_recompute, or its _fp8 forms when fp8 != 0) is expected
 * to be at least as fast as recomputing into a buffer and attending over it in two calls, for `total_rows`
 * evicted rows over all sequences of the launch; 0 otherwise or on bad arguments.  A rule fitted to
 * measurements on B200 (bf16: from 16384 rows, FP8: from 4096 rows per launch), not a guarantee. */
int kvd_fused_recompute_pays(const kvd_model_desc *desc, int64_t total_rows, int fp8);

/* The same with the evicted tokens taken from the FP8 store (kvd_checkpoint_residual_fp8): ranges[b] (HOST
 * [batch], rows of the FP8 store of (layer, ranges[b].seq); k_out / v_out ignored) are rebuilt with E4M3
 * operands and attended inside the recompute kernel.  There are no caller rows here: the new tokens are
 * quantised into the FP8 store first and either belong to ranges[b] (nothing is kept: a cache budget of
 * zero) or are listed in store_ranges (HOST [n_store_ranges], batch + n_store_ranges <=
 * KVD_MAX_STORE_RANGES), whose K and V ARE written to their k_out / v_out (row stride out_row_stride) for
 * the live segments to point at.  Result: attention over [keys of ranges[b]] united with segs[b][*], with
 * the tolerance and the definition of kvd_recompute_kv_fp8.  Shapes and attachments as above, the FP8
 * store in place of the bf16 one. */
kvd_status kvd_decode_attention_recompute_fp8(kvd_ctx *ctx, int layer, int batch, const void *q, const int32_t *q_pos,
                                              const kvd_store_range *ranges, const kvd_store_range *store_ranges,
                                              int n_store_ranges, int64_t out_row_stride, const kvd_kv_segment *segs,
                                              int n_segs, float scale, void *out, void *stream);
/* The same with caller-held quantised rows (see kvd_fp8_rows) stored next to store_ranges. */
kvd_status kvd_decode_attention_recompute_fp8_rows(kvd_ctx *ctx, int layer, int batch, const void *q,
                                                   const int32_t *q_pos, const kvd_store_range *ranges,
                                                   const kvd_store_range *store_ranges, int n_store_ranges,
                                                   const kvd_fp8_rows *rows, int64_t out_row_stride,
                                                   const kvd_kv_segment *segs, int n_segs, float scale, void *out,
                                                   void *stream);

/* No counterpart in the paper: the same decode attention as kvd_decode_attention for callers that
 * cannot allocate device memory at all -- code running inside someone else's memory pool or under a
 * fixed memory budget, a plug-in whose host forbids cudaMalloc after start-up, a process that must
 * not disturb an allocator's bookkeeping.  It needs no context and no workspace: the split partials
 * live in a fixed array of KVD_STATIC_SCRATCH_BYTES compiled into the
 * library, which every GPU that loads the library holds until the process exits.
 *   - Shapes are passed directly (d_head in {64, 128, 256}, group size n_q_heads / n_kv_heads in
 *     {1, 2, 3, 4, 8}); q, q_pos, segs, scale, out and the visibility rule are those of
 *     kvd_decode_attention; sliding_window is the layer's window (0 = global).
 *   - The result is bit-identical to kvd_decode_attention on the same inputs.
 *   - Limits: batch <= 64 and batch * n_kv_heads <= 1024; the partials of all sequences together
 *     (at most 130 chunks per sequence and KV head up to 8192 visible keys, about 592 / n_kv_heads
 *     beyond, n_q_heads * (d_head + 2) floats each) must fit
 *     the array.  A request beyond that returns KVD_ERR_CAPACITY and launches nothing.
 *   - It calls no cudaMalloc / cudaFree and no library routine that allocates.  The first call on a
 *     device looks up the array's device address (cudaGetSymbolAddress) with that device current;
 *     make that first call outside any stream capture.
 *   - All calls share the array and it keeps the previous call's contents; every call overwrites
 *     the part it reads, so nothing has to be cleared.  Calls whose kernels can overlap on one GPU
 *     (different streams, different host threads) race on the array: serialise them on one stream. */
#define KVD_STATIC_SCRATCH_BYTES (8u << 20)
kvd_status kvd_decode_attention_static(int n_q_heads, int n_kv_heads, int d_head, int sliding_window, int batch,
                                       const void *q, const int32_t *q_pos, const kvd_kv_segment *segs, int n_segs,
                                       float scale, void *out, void *stream);

/* Fill `out` with the byte counts described at kvd_mem_stats. */
kvd_status kvd_memory_stats(const kvd_ctx *ctx, kvd_mem_stats *out);

/* Wait for `stream`, read and clear the device status word.  KVD_OK, KVD_ERR_TIMEOUT, KVD_ERR_POSITION or (checking
 * build) KVD_ERR_BOUNDS. */
kvd_status kvd_poll_status(kvd_ctx *ctx, void *stream);

/* Self-test of the failure path: enqueue a one-thread kernel that waits (at most limit_ms, 1..1000)
 * on a barrier nothing ever signals.  The wait expires, the kernel returns normally and the next
 * kvd_poll_status reports KVD_ERR_TIMEOUT -- the same mechanism every pipeline wait of the recompute
 * kernel uses (its limit is 2 s, or KVD_SPIN_LIMIT_MS from the environment at kvd_create).  The device
 * stays usable. */
kvd_status kvd_selftest_wait_timeout(kvd_ctx *ctx, int limit_ms, void *stream);

/* The checking build (libkvd_check.so: the same sources compiled with -DKVD_CHECK; python -m
 * paper_2603_19664_b200.build --check).  Its kernels test the indices they derive on the device -- the job and
 * row block a tile belongs to, the rows of a store range, the slot of a residual row, the slot of an attention
 * partial -- before they use them; a failed test sets a bit of the status word and SKIPS the access (nothing
 * faults, the context stays usable), and kvd_poll_status then returns KVD_ERR_BOUNDS.  It stands in for a
 * memory checker where none can be run; the release build contains none of these tests.
 * kvd_build_has_checks: 1 in the checking build, 0 otherwise.
 * kvd_selftest_bounds_check: runs one such test on an index that is out of range by construction (no memory is
 * touched), so that a test suite can see the mechanism report; KVD_ERR_UNSUPPORTED in the release build. */
int kvd_build_has_checks(void);
kvd_status kvd_selftest_bounds_check(kvd_ctx *ctx, void *stream);

/* Diagnostic hook: attach (buf != NULL) or detach (buf == NULL) a DEVICE buffer of int64 slots that
 * kvd_recompute_kv fills with a per-tile timeline in SM clock cycles: for CTA b and its i-th tile
 * (i < 8) the 16 slots at ((b*8 + i)*16) hold
 *   0 cycles the TMA producer waited for free stages   1/2 producer first / last issue
 *   3 cycles the MMA issuer waited for data            4/5 MMA issue start / end
 *   6/7 epilogue start / end     8 cycles the row-statistics warp waited   9 its total cycles
 *   10 tile index                11 (tile 0 only) kernel start
 *   12/13 (tile 0 only) global timer in ns at kernel start / end    14 (tile 0 only) kernel end
 * A call whose grid does not fit `bytes` records nothing.  No effect on results.  Traced variants: the bf16
 * kernel, and for the Gemma-3-4B head shape (d_head 256, 2 query heads per KV head) kvd_recompute_kv_fp8 and
 * kvd_decode_attention_recompute_fp8; other variants ignore the hook. */
kvd_status kvd_set_trace(kvd_ctx *ctx, void *buf, size_t bytes);

/* Number of kernels this context has launched since creation (all entry points). */
uint64_t kvd_launch_count(const kvd_ctx *ctx);

/* Text of the last CUDA error a call on this context hit ("" if none).  Valid until the next call. */
const char *kvd_last_cuda_error(const kvd_ctx *ctx);

const char *kvd_status_string(kvd_status s);

/* Library version, "major.minor". */
const char *kvd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVD_H_ */
