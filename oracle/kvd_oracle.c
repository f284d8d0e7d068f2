/*
 * CPU oracle for the KV-Direct hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what the paper defines:
 *   - RMSNorm                      (Eq. 1-2)
 *   - key / value projections      (Eq. 4-5, reconstruction form Eq. 13-14)
 *   - rotary position encoding     (Eq. 11-12)
 *   - softmax attention, one query (Eq. 6-7)
 * plus the per-head key normalisation that the Gemma-3 / Qwen3 shaped layers apply between the
 * projection and the rotation (not part of the paper; root-mean-square norm over d_head with a
 * learned scale shared by all heads).
 *
 * Nothing here is blocked, fused or reordered: every sum runs over its index in ascending order,
 * one output element at a time, so the code can be compared with the equations by eye.  The only
 * concession to run time is an OpenMP loop over rows / heads, which does not change any result
 * because rows and heads are independent.
 *
 * This file shares no code with the CUDA path and must never be linked into it.  Only tests, the
 * smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Parity pins (see tests/test_oracle_*.py): hand-computed cases, closed forms, invariants, a
 * library matmul on the special case where the operation reduces to one, and brute force.
 * Unpinned: nothing in this file.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define KVD_ORACLE_ROPE_INTERLEAVED 0
#define KVD_ORACLE_ROPE_HALF 1

/* Eq. 2 with the customary epsilon inside the root: sqrt(mean(x^2) + eps).  eps = 0 gives Eq. 2 literally. */
static double rms_of(const double *x, int d, double eps) {
  double s = 0.0;
  for (int i = 0; i < d; ++i) s += x[i] * x[i];
  return sqrt(s / (double)d + eps);
}

/* Eq. 1: out_i = x_i / ||x||_RMS * gamma_i */
void kvd_oracle_rmsnorm(const double *x, const double *gamma, int d, double eps, double *out) {
  const double r = rms_of(x, d, eps);
  for (int i = 0; i < d; ++i) out[i] = x[i] / r * gamma[i];
}

/*
 * Eq. 11-12: rotate pair number i (0-based) of a d_head vector by the angle pos * theta^(-2i/d_head).
 * INTERLEAVED pairs channels (2i, 2i+1) as the equations print them; HALF pairs (i, i + d_head/2).
 */
void kvd_oracle_rope(double *x, int d_head, int64_t pos, double theta, int style) {
  const int half = d_head / 2;
  for (int i = 0; i < half; ++i) {
    const double phi = (double)pos * pow(theta, -2.0 * (double)i / (double)d_head);
    const double c = cos(phi), s = sin(phi);
    const int ia = (style == KVD_ORACLE_ROPE_HALF) ? i : 2 * i;
    const int ib = (style == KVD_ORACLE_ROPE_HALF) ? i + half : 2 * i + 1;
    const double a = x[ia], b = x[ib];
    x[ia] = a * c - b * s;
    x[ib] = a * s + b * c;
  }
}

/*
 * O1: K and V of n tokens from their residual rows (Eq. 13-14).
 *   X        [n, d_hidden]              residual rows entering the layer
 *   pos      [n]                        absolute position of each row
 *   gamma_in [d_hidden]                 pre-attention RMSNorm scale
 *   W_kv     [d_hidden, 2*n_kv*d_head]  row-major; columns [0, n_kv*d_head) are W_K (head-major),
 *                                       the rest W_V
 *   gamma_k  [d_head] or NULL           per-head key-norm scale (NULL: no key norm)
 *   K, V     [n, n_kv, d_head]          outputs
 */
void kvd_oracle_recompute_kv(const double *X, const int32_t *pos, int n, int d_hidden, int n_kv, int d_head,
                             const double *gamma_in, double rms_eps, const double *W_kv, const double *gamma_k,
                             double qk_eps, double theta, int rope_style, double *K, double *V) {
  const int kv_dim = n_kv * d_head;
  const int ldw = 2 * kv_dim;
#pragma omp parallel if (n >= 16)
  {
    double *xb = (double *)malloc(sizeof(double) * (size_t)d_hidden);
#pragma omp for schedule(dynamic, 4)
    for (int m = 0; m < n; ++m) {
      /* Eq. 1-2 */
      kvd_oracle_rmsnorm(X + (size_t)m * d_hidden, gamma_in, d_hidden, rms_eps, xb);
      double *k = K + (size_t)m * kv_dim;
      double *v = V + (size_t)m * kv_dim;
      /* Eq. 13-14 before the rotation: k[c] = sum_i xb[i] W_K[i,c], v[c] = sum_i xb[i] W_V[i,c].
       * The i loop is outermost so that W is walked along its rows; every output element still
       * receives its terms one at a time in ascending i, exactly as the dot product would. */
      for (int c = 0; c < kv_dim; ++c) k[c] = 0.0;
      for (int c = 0; c < kv_dim; ++c) v[c] = 0.0;
      for (int i = 0; i < d_hidden; ++i) {
        const double xi = xb[i];
        const double *wk = W_kv + (size_t)i * ldw;
        const double *wv = wk + kv_dim;
        for (int c = 0; c < kv_dim; ++c) k[c] += xi * wk[c];
        for (int c = 0; c < kv_dim; ++c) v[c] += xi * wv[c];
      }
      for (int h = 0; h < n_kv; ++h) {
        double *kh = k + (size_t)h * d_head;
        if (gamma_k != NULL) {
          const double r = rms_of(kh, d_head, qk_eps);
          for (int j = 0; j < d_head; ++j) kh[j] = kh[j] / r * gamma_k[j];
        }
        /* Eq. 13: R_p applied to the key only */
        kvd_oracle_rope(kh, d_head, (int64_t)pos[m], theta, rope_style);
      }
    }
    free(xb);
  }
}

/*
 * O2: one decode-attention step (Eq. 6-7) for one sequence.
 *   q      [n_q, d_head]      query heads (already normed and rotated to q_pos)
 *   Kcat   [n_keys, n_kv, d_head], Vcat likewise: the concatenation of all segments
 *   kpos   [n_keys]           absolute position of each key
 *   scale                     multiplies q.k (Eq. 6 uses 1/sqrt(d_head))
 *   window                    0 = global; otherwise key j is visible iff 0 <= q_pos - kpos[j] < window
 *   out    [n_q, d_head]
 * Query head h reads KV head h / (n_q / n_kv).  Keys with kpos > q_pos are never visible.
 * Returns the number of visible keys (the same for every head).
 */
int kvd_oracle_decode_attention(const double *q, int n_q, int n_kv, int d_head, int32_t q_pos, const double *Kcat,
                                const double *Vcat, const int32_t *kpos, int n_keys, double scale, int window,
                                double *out) {
  const int group = n_q / n_kv;
  int visible_count = 0;
  for (int j = 0; j < n_keys; ++j) {
    const int64_t dlt = (int64_t)q_pos - (int64_t)kpos[j];
    if (dlt >= 0 && (window == 0 || dlt < window)) ++visible_count;
  }
#pragma omp parallel for schedule(static) if ((long)n_keys * d_head >= 262144)
  for (int h = 0; h < n_q; ++h) {
    const int g = h / group;
    double *s = (double *)malloc(sizeof(double) * (size_t)(n_keys > 0 ? n_keys : 1));
    double m = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
      const int64_t dlt = (int64_t)q_pos - (int64_t)kpos[j];
      const int vis = dlt >= 0 && (window == 0 || dlt < window);
      if (!vis) {
        s[j] = -INFINITY;
        continue;
      }
      const double *kj = Kcat + ((size_t)j * n_kv + g) * d_head;
      double acc = 0.0;
      for (int c = 0; c < d_head; ++c) acc += q[(size_t)h * d_head + c] * kj[c];
      s[j] = scale * acc;
      if (s[j] > m) m = s[j];
    }
    double denom = 0.0;
    for (int c = 0; c < d_head; ++c) out[(size_t)h * d_head + c] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
      if (s[j] == -INFINITY) continue;
      const double p = exp(s[j] - m);
      denom += p;
      const double *vj = Vcat + ((size_t)j * n_kv + g) * d_head;
      for (int c = 0; c < d_head; ++c) out[(size_t)h * d_head + c] += p * vj[c];
    }
    if (denom > 0.0)
      for (int c = 0; c < d_head; ++c) out[(size_t)h * d_head + c] /= denom;
    free(s);
  }
  return visible_count;
}

int kvd_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void kvd_oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}
