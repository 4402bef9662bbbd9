/*
 * fp64 CPU oracle for SSD (Spatial-Semantic head Decoupling) KV-cache compression.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes, written from the paper.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.  It shares no code, header,
 * table or constant with the CUDA library and neither includes the other.
 *
 * All inputs are bf16 bit patterns (uint16) -- the very tensors the GPU path
 * receives -- widened exactly to double; all arithmetic is double; softmax is
 * computed by subtracting the row maximum.
 *
 * Notation (paper, Sec. 3.1): L prompt tokens, N = h*w image tokens, image step
 * t = 1..N produces image token index t-1 at absolute position L+t-1.  D is the
 * head dimension.  W, M, R are the spatial window, the semantic top-M budget and
 * the semantic reserved recent window (Sec. 3.3); w is the recency window of
 * the sparsity metric and tau its threshold (Sec. 3.3).
 *
 * Parity status: every function below is pinned by the CPU test-suite against
 * closed forms, brute force, special cases or a library routine (masked scaled
 * dot-product attention in fp64).  Nothing here is "parity unpinned".  What is
 * not pinned is fidelity to the authors' unpublished code where the paper is
 * ambiguous; those readings are parameters of these functions.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double widen(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* -------------------------------------------------------------------------
 * Attention distribution of one query over a causal context (Sec. 3.1: each
 * token is predicted from the prompt and all earlier visual tokens; standard
 * scaled dot-product softmax).
 *   q      [D]           bf16
 *   K      [n_ctx][D]    bf16, rows = absolute positions 0..n_ctx-1
 *   a_out  [n_ctx]       a_out[i] = exp(x_i - max x) / sum_j exp(x_j - max x),
 *                        x_i = scale * <q, K_i>
 * ------------------------------------------------------------------------- */
void ssd_oracle_attention_row(const uint16_t *q, const uint16_t *K, int n_ctx, int D,
                              double scale, double *a_out) {
  double xmax = -INFINITY;
  for (int i = 0; i < n_ctx; ++i) {
    double dot = 0.0;
    for (int d = 0; d < D; ++d) dot += widen(q[d]) * widen(K[(size_t)i * D + d]);
    a_out[i] = scale * dot;
    if (a_out[i] > xmax) xmax = a_out[i];
  }
  double z = 0.0;
  for (int i = 0; i < n_ctx; ++i) {
    a_out[i] = exp(a_out[i] - xmax);
    z += a_out[i];
  }
  for (int i = 0; i < n_ctx; ++i) a_out[i] /= z;
}

/* -------------------------------------------------------------------------
 * Sparsity metric, inner double sum for ONE (layer, head, prompt p)
 * (Sec. 3.3, unnumbered equation for s_{l,h}):
 *     sum_{t=1..N}  [ sum_{i=0}^{t-1-w} a_t(i) ] / [ sum_{i=0}^{t-1} a_t(i) ]
 * Reading: i indexes VISUAL tokens (i = t-1 is the query's own token); a_t is
 * the softmax over the whole causal context, prompt included, so the ratio
 * renormalises over the visual part.  Steps with t-1-w < 0 have an empty
 * numerator and contribute 0 but still count in the 1/T average.
 *   Q [N][D]      queries of image steps 1..N
 *   K [L+N][D]    keys of the prompt then the image tokens
 * ------------------------------------------------------------------------- */
double ssd_oracle_sparsity_sum(const uint16_t *Q, const uint16_t *K, int L, int N, int D, int w,
                               double scale) {
  double *a = (double *)malloc(sizeof(double) * (size_t)(L + N));
  double total = 0.0;
  for (int t = 1; t <= N; ++t) {
    ssd_oracle_attention_row(Q + (size_t)(t - 1) * D, K, L + t, D, scale, a);
    double num = 0.0, den = 0.0;
    for (int i = 0; i <= t - 1 - w; ++i) num += a[L + i];
    for (int i = 0; i <= t - 1; ++i) den += a[L + i];
    total += num / den;
  }
  free(a);
  return total;
}

/* s_{l,h} = (1/P) sum_p (1/T) sum_t ratio, T = N (Sec. 3.3).
 *   Q_cal [n_layers][P][H][N][D], K_cal [n_layers][P][H][L+N][D]
 *   s_out [n_layers][H]
 */
void ssd_oracle_sparsity(const uint16_t *Q_cal, const uint16_t *K_cal, int n_layers, int P, int H,
                         int L, int N, int D, int w, double scale, double *s_out) {
  double *part = (double *)malloc(sizeof(double) * (size_t)n_layers * P * H);
#pragma omp parallel for schedule(dynamic, 1)
  for (long u = 0; u < (long)n_layers * P * H; ++u) {
    part[u] = ssd_oracle_sparsity_sum(Q_cal + (size_t)u * N * D, K_cal + (size_t)u * (L + N) * D,
                                      L, N, D, w, scale);
  }
  for (int l = 0; l < n_layers; ++l)
    for (int h = 0; h < H; ++h) {
      double acc = 0.0;
      for (int p = 0; p < P; ++p) acc += part[((size_t)l * P + p) * H + h];
      s_out[(size_t)l * H + h] = acc / ((double)P * (double)N);
    }
  free(part);
}

/* Head type (Sec. 3.3, threshold equation): Semantic iff s > tau; s == tau is
 * Spatial.  label 1 = Semantic, 0 = Spatial. */
void ssd_oracle_labels(const double *s, int n, double tau, uint8_t *label_out) {
  for (int i = 0; i < n; ++i) label_out[i] = (s[i] > tau) ? 1 : 0;
}

/* -------------------------------------------------------------------------
 * Accumulated attention score of each image token for ONE (sequence, head)
 * (Algorithm 1, the AttentionScores / running-sum lines):
 *     score[j] = sum over observed steps t with t-1 >= j of a_t(L+j)
 * observed steps are t = n0-n_obs+1 .. n0; a_t is post-softmax over the whole
 * causal context (prompt included).  n_obs = n0 is the paper's running sum.
 *   Q_obs [n_obs][D]   row r is the query of image step n0-n_obs+1+r
 *   K     [L+n0][D]
 *   score_out [n0]
 *   prompt_mass_out (may be NULL): total probability the observed rows put on
 *   the L prompt positions (so that sum(score)+prompt_mass = n_obs).
 * ------------------------------------------------------------------------- */
void ssd_oracle_scores(const uint16_t *Q_obs, const uint16_t *K, int L, int n0, int n_obs, int D,
                       double scale, double *score_out, double *prompt_mass_out) {
  double *a = (double *)malloc(sizeof(double) * (size_t)(L + n0 + 1));
  double pm = 0.0;
  for (int j = 0; j < n0; ++j) score_out[j] = 0.0;
  for (int r = 0; r < n_obs; ++r) {
    int t = n0 - n_obs + 1 + r;
    ssd_oracle_attention_row(Q_obs + (size_t)r * D, K, L + t, D, scale, a);
    for (int j = 0; j <= t - 1; ++j) score_out[j] += a[L + j];
    for (int i = 0; i < L; ++i) pm += a[i];
  }
  if (prompt_mass_out) *prompt_mass_out = pm;
  free(a);
}

/* -------------------------------------------------------------------------
 * IndicesOfTopM (Algorithm 1).  Candidates are image indices 0..n_cand-1 (the
 * caller passes n_cand = max(0, n0-R): the R newest tokens are reserved, not
 * candidates).  Picks min(M, n_cand) largest scores; among equal scores the
 * lowest index wins; result ascending.  Returns the count.
 * ------------------------------------------------------------------------- */
int ssd_oracle_topm(const double *score, int n_cand, int M, int32_t *idx_out) {
  int k = M < n_cand ? M : n_cand;
  if (k <= 0) return 0;
  uint8_t *taken = (uint8_t *)calloc((size_t)n_cand, 1);
  for (int s = 0; s < k; ++s) {
    int best = -1;
    for (int j = 0; j < n_cand; ++j) {
      if (taken[j]) continue;
      if (best < 0 || score[j] > score[best]) best = j; /* strict > keeps lowest index */
    }
    taken[best] = 1;
  }
  int c = 0;
  for (int j = 0; j < n_cand; ++j)
    if (taken[j]) idx_out[c++] = j;
  free(taken);
  return c;
}

/* -------------------------------------------------------------------------
 * Retained set of one head after image token t-1 has been appended (Sec. 3.3
 * policies; Algorithm 1 spatial and semantic branches).  Absolute positions,
 * ascending, no duplicates.  Returns the count.
 *   spatial : {0..L-1} U {L+j : max(0,t-W) <= j <= t-1}
 *   semantic: {0..L-1} U {L+j : j in top_idx} U {L+j : max(0,t-R) <= j <= t-1}
 * The window sizes INCLUDE the newest token (fixed-size cache).
 * ------------------------------------------------------------------------- */
int ssd_oracle_retained_set(int is_semantic, int L, int t, int W, int R, const int32_t *top_idx,
                            int n_top, int32_t *pos_out) {
  int n = 0;
  for (int i = 0; i < L; ++i) pos_out[n++] = i;
  int cap = is_semantic ? R : W;
  int lo = t - cap > 0 ? t - cap : 0;
  if (is_semantic)
    for (int k = 0; k < n_top; ++k)
      if (top_idx[k] < lo) pos_out[n++] = L + top_idx[k]; /* guard only against overlap */
  for (int j = lo; j <= t - 1; ++j) pos_out[n++] = L + j;
  return n;
}

/* -------------------------------------------------------------------------
 * Attention of one query restricted to a set of positions (the consumer of
 * Algorithm 1's output):  out = sum_i softmax_i(scale <q,K_pos[i]>) V_pos[i].
 *   K_hist, V_hist [n_hist][D]  full uncompressed history, indexed by position
 *   pos [n_pos]                 positions to attend to
 *   out [D]; weights_out [n_pos] may be NULL
 * ------------------------------------------------------------------------- */
void ssd_oracle_attend(const uint16_t *q, const uint16_t *K_hist, const uint16_t *V_hist, int D,
                       const int32_t *pos, int n_pos, double scale, double *out,
                       double *weights_out) {
  double *x = (double *)malloc(sizeof(double) * (size_t)(n_pos > 0 ? n_pos : 1));
  double xmax = -INFINITY;
  for (int i = 0; i < n_pos; ++i) {
    double dot = 0.0;
    const uint16_t *k = K_hist + (size_t)pos[i] * D;
    for (int d = 0; d < D; ++d) dot += widen(q[d]) * widen(k[d]);
    x[i] = scale * dot;
    if (x[i] > xmax) xmax = x[i];
  }
  double z = 0.0;
  for (int i = 0; i < n_pos; ++i) {
    x[i] = exp(x[i] - xmax);
    z += x[i];
  }
  for (int d = 0; d < D; ++d) out[d] = 0.0;
  for (int i = 0; i < n_pos; ++i) {
    double p = x[i] / z;
    if (weights_out) weights_out[i] = p;
    const uint16_t *v = V_hist + (size_t)pos[i] * D;
    for (int d = 0; d < D; ++d) out[d] += p * widen(v[d]);
  }
  free(x);
}

/* -------------------------------------------------------------------------
 * Batched drivers (plain loops over independent (sequence, head) pairs, spread
 * over host threads; no arithmetic of their own).
 * ------------------------------------------------------------------------- */

/* Scores + selection for a batch of pairs.
 *   Q_obs [n_pairs][n_obs][D], K [n_pairs][L+n_keys][D] (n_keys >= n0 image rows present)
 *   is_semantic [n_pairs]; score_out [n_pairs][n0] (zeros for spatial pairs)
 *   idx_out [n_pairs][M] (-1 padded); cnt_out [n_pairs]
 */
void ssd_oracle_select_batch(const uint16_t *Q_obs, const uint16_t *K, const uint8_t *is_semantic,
                             long n_pairs, int L, int n_keys, int n0, int n_obs, int D, int M, int R,
                             double scale, double *score_out, int32_t *idx_out, int32_t *cnt_out) {
#pragma omp parallel for schedule(dynamic, 1)
  for (long u = 0; u < n_pairs; ++u) {
    double *sc = score_out + (size_t)u * n0;
    int32_t *ix = idx_out + (size_t)u * M;
    for (int m = 0; m < M; ++m) ix[m] = -1;
    for (int j = 0; j < n0; ++j) sc[j] = 0.0;
    cnt_out[u] = 0;
    if (!is_semantic[u]) continue;
    ssd_oracle_scores(Q_obs + (size_t)u * n_obs * D, K + (size_t)u * (L + n_keys) * D, L, n0, n_obs,
                      D, scale, sc, NULL);
    int n_cand = n0 - R > 0 ? n0 - R : 0;
    cnt_out[u] = ssd_oracle_topm(sc, n_cand, M, ix);
  }
}

/* Decode attention at image step t for a batch of pairs.
 *   q [n_pairs][D]; K_hist, V_hist [n_pairs][L+n_keys][D] with n_keys >= t
 *   idx [n_pairs][M], cnt [n_pairs] from the selection; out [n_pairs][D]
 *   full != 0 ignores the policies and attends to all positions 0..L+t-1.
 */
void ssd_oracle_decode_batch(const uint16_t *q, const uint16_t *K_hist, const uint16_t *V_hist,
                             const uint8_t *is_semantic, const int32_t *idx, const int32_t *cnt,
                             long n_pairs, int L, int n_keys, int t, int D, int W, int M, int R,
                             double scale, int full, double *out) {
#pragma omp parallel for schedule(dynamic, 4)
  for (long u = 0; u < n_pairs; ++u) {
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + t + M + 1));
    int n;
    if (full) {
      n = L + t;
      for (int i = 0; i < n; ++i) pos[i] = i;
    } else {
      n = ssd_oracle_retained_set(is_semantic[u], L, t, W, R, idx ? idx + (size_t)u * M : NULL,
                                  cnt ? cnt[u] : 0, pos);
    }
    ssd_oracle_attend(q + (size_t)u * D, K_hist + (size_t)u * (L + n_keys) * D,
                      V_hist + (size_t)u * (L + n_keys) * D, D, pos, n, scale, out + (size_t)u * D,
                      NULL);
    free(pos);
  }
}

#ifdef _OPENMP
#include <omp.h>
int ssd_oracle_threads(void) { return omp_get_max_threads(); }
#else
int ssd_oracle_threads(void) { return 1; }
#endif
