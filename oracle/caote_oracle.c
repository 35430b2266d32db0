/*
 * caote_oracle.c — TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, double-precision CPU statement of what the CAOTE eviction-scoring attention step
 * computes, written from the paper's equations. It exists so that the CUDA library can be checked
 * against something that is easy to verify by eye. It shares no code with the CUDA path, and only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Everything is computed in double from the caller's values exactly as given (bf16/fp32 inputs are
 * widened by the caller, which is exact). There is no blocking, no fusion and no reordering beyond
 * what the equations state. OpenMP, when enabled, only spreads independent (unit, query head) pairs
 * over threads; the per-head partial sums are then added in a fixed order.
 *
 * Layout (row-major): q [B, Hq, m, d]; K, V [B, Hkv, cap, d]; base, scores, w [B, Hkv, cap];
 * o [B, Hq, m, d]; X [B, Hkv, d]; len [B]. Query head hq belongs to KV head hq / G, G = Hq / Hkv.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { BASE_LAST_QUERY = 0, BASE_CHUNK_SUM = 1, BASE_ACCUM = 2, BASE_EXTERNAL = 3 };
enum { AGG_WEIGHTS = 0, AGG_SUM_ERRORS = 1 };

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim, capacity, n_new;
  double scale;
  int32_t base_mode, agg_mode;
} oracle_params_t;

/* Softmax attention of ONE query row over its first n_vis cached tokens (Sec. 2, generation
 * equation: A = Softmax(q [K_{:t}, k_new]^T), X_attn = A V; the explicit logit scale is this
 * build's reading, the paper writes none).
 *   alpha[j] (j < n_vis) and o[c] (c < d) out. */
static void attention_row(const float* q, const float* K, const float* V, int n_vis, int d,
                          double scale, double* alpha, double* o) {
  double smax = -INFINITY;
  for (int j = 0; j < n_vis; ++j) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += (double)q[c] * (double)K[(size_t)j * d + c];
    s *= scale;
    alpha[j] = s;
    if (s > smax) smax = s;
  }
  double denom = 0.0;
  for (int j = 0; j < n_vis; ++j) {
    alpha[j] = exp(alpha[j] - smax);
    denom += alpha[j];
  }
  for (int j = 0; j < n_vis; ++j) alpha[j] /= denom;
  for (int c = 0; c < d; ++c) o[c] = 0.0;
  for (int j = 0; j < n_vis; ++j)
    for (int c = 0; c < d; ++c) o[c] += alpha[j] * (double)V[(size_t)j * d + c];
}

/* || x - v ||_2 over d channels (Sec. 3.1: any norm could be used, the paper picks L2; the text's
 * "mean square error" is read as this un-squared, un-averaged norm, as every formula writes it). */
static double l2_distance(const double* x, const float* v, int d) {
  double acc = 0.0;
  for (int c = 0; c < d; ++c) {
    double t = x[c] - (double)v[c];
    acc += t * t;
  }
  return sqrt(acc);
}

/* CAOTE score of every token from non-negative base scores h (Sec. 3.2 general form):
 *   w_j = h_j / sum_i h_i,  X = sum_j w_j v_j,  c_j = w_j / (1 - w_j) * || X - v_j ||_2.
 * 1 - w_j is formed as (sum_{i != j} h_i) / (sum_i h_i), a sum of non-negative terms, so that a
 * token holding almost all the weight does not lose its score to cancellation.
 * Readings where the paper is silent: sum h == 0 gives c = 0 for all; a token whose complement is
 * exactly 0 (it holds all the weight, e.g. n == 1) gets +inf (never the first to go). */
static void caote_from_base(const double* h, const float* V, int n, int d, double* w, double* X,
                            double* c) {
  double* prefix = (double*)malloc(sizeof(double) * (size_t)(n + 1));
  double* suffix = (double*)malloc(sizeof(double) * (size_t)(n + 1));
  prefix[0] = 0.0;
  for (int j = 0; j < n; ++j) prefix[j + 1] = prefix[j] + h[j];
  suffix[n] = 0.0;
  for (int j = n - 1; j >= 0; --j) suffix[j] = suffix[j + 1] + h[j];
  const double total = prefix[n];
  for (int cc = 0; cc < d; ++cc) X[cc] = 0.0;
  if (!(total > 0.0)) {
    for (int j = 0; j < n; ++j) {
      w[j] = 0.0;
      c[j] = 0.0;
    }
    free(prefix);
    free(suffix);
    return;
  }
  for (int j = 0; j < n; ++j) {
    w[j] = h[j] / total;
    for (int cc = 0; cc < d; ++cc) X[cc] += w[j] * (double)V[(size_t)j * d + cc];
  }
  for (int j = 0; j < n; ++j) {
    const double rest = (prefix[j] + suffix[j + 1]) / total; /* 1 - w_j */
    if (rest == 0.0)
      c[j] = INFINITY;
    else
      c[j] = w[j] / rest * l2_distance(X, V + (size_t)j * d, d);
  }
  free(prefix);
  free(suffix);
}

/* The scoring step for all units.
 *   base: in/out for ACCUM (this call's attention mass is added first, then h = base), in for
 *         EXTERNAL, unused otherwise (may be NULL).
 *   o, scores: out.  w, X: optional outputs (NULL to skip).  scores / w of slots >= len[b] are
 *   left untouched. Sequences with len[b] == 0 are skipped.
 * agg_mode AGG_WEIGHTS: base scores of the G heads (and of the block's rows) are added, then the
 *   general form is applied once per unit (this build's reading of how the single-head, single-query
 *   derivation extends to grouped-query attention and to a block of queries: Sec. 2 f_score
 *   aggregates rows first; the K/V rows are shared by the group, so eviction is per KV head).
 * agg_mode AGG_SUM_ERRORS: c_j = sum over the rows that define the base score of the exact
 *   single-query error alpha/(1-alpha) * ||o_row - v_j|| (Theorem 3.2 applied row by row). Only
 *   defined for LAST_QUERY and CHUNK_SUM.
 * Returns 0, or -1 on a bad argument. */
int caote_oracle_score(const oracle_params_t* p, const float* q, const float* K, const float* V,
                       const int32_t* len, double* base, double* o, double* scores, double* w_out,
                       double* X_out) {
  const int B = p->batch, Hq = p->n_q_heads, Hkv = p->n_kv_heads, d = p->head_dim;
  const int cap = p->capacity, m = p->n_new;
  if (B < 1 || Hkv < 1 || Hq % Hkv != 0 || d < 1 || m < 1 || cap < 1) return -1;
  if ((p->base_mode == BASE_ACCUM || p->base_mode == BASE_EXTERNAL) && base == NULL) return -1;
  if (p->agg_mode == AGG_SUM_ERRORS && p->base_mode != BASE_LAST_QUERY &&
      p->base_mode != BASE_CHUNK_SUM)
    return -1;
  const int G = Hq / Hkv;
  for (int b = 0; b < B; ++b)
    if (len[b] != 0 && (len[b] < m || len[b] > cap)) return -1;

  /* per (unit, group head): this call's attention mass per token, and the summed per-row errors */
  const size_t units = (size_t)B * Hkv;
  double* mass = (double*)calloc(units * G * cap, sizeof(double));
  double* err = (double*)calloc(units * G * cap, sizeof(double));
  if (!mass || !err) return -1;

#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (long u = 0; u < (long)units; ++u) {
    for (int g = 0; g < G; ++g) {
      const int b = (int)(u / Hkv), h = (int)(u % Hkv);
      const int n = len[b];
      if (n == 0) continue;
      const float* Ku = K + (size_t)u * cap * d;
      const float* Vu = V + (size_t)u * cap * d;
      const int hq = h * G + g;
      double* alpha = (double*)malloc(sizeof(double) * (size_t)n);
      double* mrow = mass + (u * G + g) * cap;
      double* erow = err + (u * G + g) * cap;
      for (int i = 0; i < m; ++i) {
        const int n_vis = n - m + i + 1; /* query i sees slots 0 .. n-m+i (causal inside the block) */
        const float* qi = q + (((size_t)b * Hq + hq) * m + i) * d;
        double* oi = o + (((size_t)b * Hq + hq) * m + i) * d;
        attention_row(qi, Ku, Vu, n_vis, d, p->scale, alpha, oi);
        const int counted = (p->base_mode == BASE_LAST_QUERY) ? (i == m - 1) : 1;
        if (!counted) continue;
        for (int j = 0; j < n_vis; ++j) {
          mrow[j] += alpha[j];
          /* Sec. 3.1 CAOTE score of token j for this single query row; 1 - alpha_j as the sum of
           * the other weights */
          double rest = 0.0;
          if (p->agg_mode == AGG_SUM_ERRORS) {
            for (int t = 0; t < n_vis; ++t)
              if (t != j) rest += alpha[t];
            erow[j] += (rest == 0.0) ? INFINITY
                                     : alpha[j] / rest * l2_distance(oi, Vu + (size_t)j * d, d);
          }
        }
      }
      free(alpha);
    }
  }

  for (size_t u = 0; u < units; ++u) {
    const int b = (int)(u / Hkv);
    const int n = len[b];
    if (n == 0) continue;
    const float* Vu = V + u * cap * d;
    double* hvec = (double*)malloc(sizeof(double) * (size_t)n);
    double* wvec = (double*)malloc(sizeof(double) * (size_t)n);
    double* Xvec = (double*)malloc(sizeof(double) * (size_t)d);
    for (int j = 0; j < n; ++j) {
      double s = 0.0;
      for (int g = 0; g < G; ++g) s += mass[(u * G + g) * cap + j];
      switch (p->base_mode) {
        case BASE_ACCUM:
          base[u * cap + j] += s; /* Sec. 3.2 "CAOTE for H2O": sum of all attention given to j */
          hvec[j] = base[u * cap + j];
          break;
        case BASE_EXTERNAL:
          hvec[j] = base[u * cap + j];
          break;
        default:
          hvec[j] = s;
      }
    }
    caote_from_base(hvec, Vu, n, d, wvec, Xvec, scores + u * cap);
    if (p->agg_mode == AGG_SUM_ERRORS) {
      for (int j = 0; j < n; ++j) {
        double s = 0.0;
        for (int g = 0; g < G; ++g) s += err[(u * G + g) * cap + j];
        scores[u * cap + j] = s;
      }
    }
    if (w_out) memcpy(w_out + u * cap, wvec, sizeof(double) * (size_t)n);
    if (X_out) memcpy(X_out + u * d, Xvec, sizeof(double) * (size_t)d);
    free(hvec);
    free(wvec);
    free(Xvec);
  }
  free(mass);
  free(err);
  return 0;
}

/* FastCAOTE (Sec. 3.3): the same score with X replaced by the plain mean of the n cached values.
 * w in (already normalised weights, e.g. the w output of caote_oracle_score); c out. One unit. */
void caote_oracle_fast_scores(const double* w, const float* V, int n, int d, double* c) {
  double* mean = (double*)calloc((size_t)d, sizeof(double));
  for (int j = 0; j < n; ++j)
    for (int cc = 0; cc < d; ++cc) mean[cc] += (double)V[(size_t)j * d + cc];
  for (int cc = 0; cc < d; ++cc) mean[cc] /= (double)n;
  for (int j = 0; j < n; ++j) {
    double rest = 0.0;
    for (int t = 0; t < n; ++t)
      if (t != j) rest += w[t];
    c[j] = (rest == 0.0) ? INFINITY : w[j] / rest * l2_distance(mean, V + (size_t)j * d, d);
  }
  free(mean);
}

/* Joint error of evicting a set E of tokens at once (Appendix B, multi-token equation):
 *   c_E = || sum_{i in E} w_i (X - v_i) ||_2 / (1 - sum_{i in E} w_i),  X = sum_j w_j v_j.
 * One unit; w are normalised weights; E holds n_e distinct slot indices. */
double caote_oracle_joint_score(const double* w, const float* V, int n, int d, const int32_t* E,
                                int n_e) {
  double* X = (double*)calloc((size_t)d, sizeof(double));
  double* acc = (double*)calloc((size_t)d, sizeof(double));
  for (int j = 0; j < n; ++j)
    for (int c = 0; c < d; ++c) X[c] += w[j] * (double)V[(size_t)j * d + c];
  double gone = 0.0;
  for (int e = 0; e < n_e; ++e) {
    const int j = E[e];
    gone += w[j];
    for (int c = 0; c < d; ++c) acc[c] += w[j] * (X[c] - (double)V[(size_t)j * d + c]);
  }
  double nrm = 0.0;
  for (int c = 0; c < d; ++c) nrm += acc[c] * acc[c];
  free(X);
  free(acc);
  return sqrt(nrm) / (1.0 - gone);
}

/* Greedy multi-token eviction (Appendix B, the two-token derivation chained k times): evict one token,
 * renormalise what is left, evict the next one from the updated state.
 *   repeat k times over the tokens still present:
 *     c_j = w_j / (1 - w_j) * || X - v_j ||_2 on the CURRENT weights and output (Sec. 3.1 score; 1 - w_j
 *           as the sum of the other present weights);
 *     e   = the present token with the smallest (c_j, pos_j) (pos == NULL: the slot index);
 *     X  <- (X - w_e v_e) / (1 - w_e),  w_i <- w_i / (1 - w_e) for the others   (Appendix B, alpha' and X').
 * One unit. w in: normalised weights of the n tokens (sum 1). Outputs: order[t] = slot evicted at step t,
 * step_score[t] = its score at that step (the output error of that single step), cum_err[t] = the distance
 * between the ORIGINAL output and the output after t + 1 evictions (which the closed-form joint score of
 * Appendix B gives for the evicted set). Any output may be NULL. k < n required. Returns 0, or -1. */
int caote_oracle_greedy_evict(const double* w_in, const float* V, const int32_t* pos, int n, int d, int k,
                              int32_t* order, double* step_score, double* cum_err) {
  if (n < 1 || d < 1 || k < 0 || k >= n) return -1;
  double* w = (double*)malloc(sizeof(double) * (size_t)n);
  char* present = (char*)malloc((size_t)n);
  double* X = (double*)calloc((size_t)d, sizeof(double));
  double* X0 = (double*)malloc(sizeof(double) * (size_t)d);
  for (int j = 0; j < n; ++j) {
    w[j] = w_in[j];
    present[j] = 1;
    for (int c = 0; c < d; ++c) X[c] += w[j] * (double)V[(size_t)j * d + c];
  }
  memcpy(X0, X, sizeof(double) * (size_t)d);
  for (int t = 0; t < k; ++t) {
    int best = -1;
    double best_c = 0.0;
    for (int j = 0; j < n; ++j) {
      if (!present[j]) continue;
      double rest = 0.0;
      for (int i = 0; i < n; ++i)
        if (present[i] && i != j) rest += w[i];
      const double c = (rest == 0.0) ? INFINITY : w[j] / rest * l2_distance(X, V + (size_t)j * d, d);
      const int pj = pos ? pos[j] : j;
      if (best < 0 || c < best_c || (c == best_c && pj < (pos ? pos[best] : best))) {
        best = j;
        best_c = c;
      }
    }
    const double we = w[best];
    double rest = 0.0;
    for (int i = 0; i < n; ++i)
      if (present[i] && i != best) rest += w[i];
    present[best] = 0;
    for (int c = 0; c < d; ++c) X[c] = (X[c] - we * (double)V[(size_t)best * d + c]) / rest;
    for (int i = 0; i < n; ++i)
      if (present[i]) w[i] /= rest;
    if (order) order[t] = best;
    if (step_score) step_score[t] = best_c;
    if (cum_err) {
      double acc = 0.0;
      for (int c = 0; c < d; ++c) acc += (X0[c] - X[c]) * (X0[c] - X[c]);
      cum_err[t] = sqrt(acc);
    }
  }
  free(w);
  free(present);
  free(X);
  free(X0);
  return 0;
}
