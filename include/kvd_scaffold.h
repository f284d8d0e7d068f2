/*
 * kvd_scaffold.h -- the parts of a decoder layer AROUND the KV-Direct hot path, for tests and benchmarks.
 *
 * kvd.h is the library: checkpoint, recompute, decode attention.  To run Algorithm 1 of the paper on a whole
 * decoder stack -- which the token-identity experiments and the decode-step timings need -- something also has
 * to compute the query projection (Eq. 3), the output projection and residual add (Eq. 8), the MLP and its
 * residual add (Eq. 9), the final norm, the vocabulary projection and the greedy pick.  None of that is part of
 * the method, and both cache policies share every bit of it; it is scaffolding.  These entry points provide it
 * on the library's own kernels, so that a whole-stack run uses no third-party GEMM or elementwise library:
 *
 *   kvd_scaffold_linear          out = s (x W'),  W' = diag(gamma) W prepared once; s = 1/rms(x) per row when a
 *                                gamma was given (RMSNorm of Eq. 1-2 folded in), 1 otherwise.  Runs on the
 *                                recompute kernel of kvd.h (same tcgen05 tiles, every column treated as a value
 *                                column), so a row's output bits do not depend on how many rows a call carries.
 *   kvd_scaffold_query_finish    per query head: optional RMS norm over d_head, then the rotation of Eq. 11-12
 *                                at the row's position (the same tables as the keys).
 *   kvd_scaffold_add_rows        h <- h + y (Eq. 8 / Eq. 9 residual adds), rounded to bf16.
 *   kvd_scaffold_gated_act       act(gate) * up of a gated MLP (tanh-GELU or SiLU).
 *   kvd_scaffold_embed           gather rows of the embedding table.
 *   kvd_scaffold_argmax          greedy pick: index of the largest logit per row, lowest index on ties.
 *
 * Conventions are those of kvd.h: plain C, DEVICE pointers are the caller's bf16 buffers (16-byte aligned),
 * launches are asynchronous on `stream`, argument errors are found on the host before anything is launched,
 * bf16 contexts only (KVD_ERR_UNSUPPORTED after kvd_set_dtype chose another type).  Throughput is not the
 * point of these calls: a product always walks 256-row tiles, whatever the batch.
 */
#ifndef KVD_SCAFFOLD_H_
#define KVD_SCAFFOLD_H_

#include "kvd.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvd_linear kvd_linear; /* opaque: one prepared weight matrix */

#define KVD_ACT_GELU_TANH 0
#define KVD_ACT_SILU 1

/* Prepare out = s (x W') for w DEVICE bf16 [k, n] row-major (k % 64 == 0).  gamma DEVICE bf16 [k] or NULL:
 * with a gamma, W' = diag(gamma) W and every row is scaled by 1/sqrt(mean(x^2) + rms_eps) (Eq. 1-2 ahead of
 * the product); without, W' = W and s = 1.  The prepared copy (bf16, K-major, n rounded up to the tile width
 * with zero columns) is owned by the handle.  Enqueues on `stream` and waits for it. */
kvd_status kvd_scaffold_linear_create(kvd_ctx *ctx, const void *w, const void *gamma, int k, int n, float rms_eps,
                                      void *stream, kvd_linear **out);
void kvd_scaffold_linear_destroy(kvd_ctx *ctx, kvd_linear *lin);

/* Columns a call writes per row: n rounded up to a multiple of the tile width (128 or 256); columns >= n are
 * written as zeros.  `out` of kvd_scaffold_linear needs a row stride of at least this many elements. */
int kvd_scaffold_linear_out_cols(const kvd_linear *lin);

/* out[m, :] = s_m (x[m, :] W') for x DEVICE bf16 [m, k] (contiguous rows); out DEVICE bf16, row stride
 * out_row_stride elements (multiple of 8, >= kvd_scaffold_linear_out_cols).  One launch (two when m > 64 and
 * the product is normalised: the rows' statistics first).  KVD_ERR_CAPACITY when m exceeds
 * max_seqs * max_tokens_per_seq of the context. */
kvd_status kvd_scaffold_linear(kvd_ctx *ctx, const kvd_linear *lin, const void *x, int m, void *out,
                               int64_t out_row_stride, void *stream);

/* Queries of `layer` from their raw projection: q_in DEVICE bf16, row r head h channel c at
 * q_in[r * in_row_stride + h * d_head + c]; per head, when gamma_q != NULL (DEVICE bf16 [d_head]),
 * q <- q / sqrt(mean_c q_c^2 + qk_norm_eps) * gamma_q, then the rotation R_pos of Eq. 11-12 with the layer's
 * theta and the context's pairing; positions DEVICE int32 [m].  q_out DEVICE bf16 [m, n_q_heads, d_head],
 * the layout kvd_decode_attention expects. */
kvd_status kvd_scaffold_query_finish(kvd_ctx *ctx, int layer, const void *q_in, int64_t in_row_stride,
                                     const int32_t *positions, int m, const void *gamma_q, void *q_out, void *stream);

/* h[r, c] <- bf16(h[r, c] + y[r * y_row_stride + c]) for r < m, c < d (d % 8 == 0). */
kvd_status kvd_scaffold_add_rows(kvd_ctx *ctx, void *h, const void *y, int64_t y_row_stride, int m, int d,
                                 void *stream);

/* out[r, c] = bf16(act(gate_up[r * row_stride + c]) * gate_up[r * row_stride + width + c]) for c < width
 * (width % 8 == 0): the inner product of a gated MLP whose gate and up projections were computed as one
 * [k, 2 * width] product.  activation: KVD_ACT_GELU_TANH or KVD_ACT_SILU.  out DEVICE bf16 [m, width]. */
kvd_status kvd_scaffold_gated_act(kvd_ctx *ctx, const void *gate_up, int64_t row_stride, int m, int width,
                                  int activation, void *out, void *stream);

/* out[r, :] = table[tokens[r], :]; table DEVICE bf16 [vocab, d] (d % 8 == 0), tokens DEVICE int32 [m].  A token
 * outside [0, vocab) reads row 0 and sets the position bit of the status word (kvd_poll_status). */
kvd_status kvd_scaffold_embed(kvd_ctx *ctx, const void *table, const int32_t *tokens, int m, int d, int vocab,
                              void *out, void *stream);

/* tokens_out[r] = argmax_c logits[r * row_stride + c] over c < n, the lowest index among equal maxima
 * (NaNs never win; a row of NaNs yields 0).  logits DEVICE bf16; tokens_out DEVICE int32 [m].  Two small launches
 * and a memset of a per-row slot owned by the context (allocated on first use: make the first call outside stream
 * capture). */
kvd_status kvd_scaffold_argmax(kvd_ctx *ctx, const void *logits, int64_t row_stride, int m, int n,
                               int32_t *tokens_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* KVD_SCAFFOLD_H_ */
