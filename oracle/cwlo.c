/*
 * cwlo.c -- fp64 CPU oracle for the ChunkWise-LoRA hot path (TEST INFRASTRUCTURE ONLY).
 * See cwlo.h for scope, citations and pin status.  No blocking, no fusion, no BLAS: every
 * function is the definition (or the algorithm's steps in order) written out.
 */
#include "cwlo.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define Q24 16777216 /* 2^24 */

int cwlo_get_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void cwlo_set_threads(int n) {
#ifdef _OPENMP
  if (n >= 1) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* ---------------------------------------------------------------------------------------------
 * Sec. III-A signal (i): next-token entropy of softmax(z), normalised by ln V so that the
 * thresholds of the selector live in [0,1].
 *   m = max z;  S = sum exp(z-m);  U = sum (z-m) exp(z-m);  H = ln S - U/S;  score = H / ln V.
 * A -inf logit has probability zero and contributes nothing.  A row holding NaN or +inf, or
 * made of -inf only, has no defined entropy: NaN (the chunker treats NaN as hardest).
 * ------------------------------------------------------------------------------------------- */
static double entropy_row(const float* z, int32_t V) {
  double m = -INFINITY;
  for (int32_t v = 0; v < V; ++v) {
    double zv = (double)z[v];
    if (isnan(zv) || zv == INFINITY) return NAN;
    if (zv > m) m = zv;
  }
  if (m == -INFINITY) return NAN;
  double S = 0.0, U = 0.0;
  for (int32_t v = 0; v < V; ++v) {
    double zv = (double)z[v];
    if (zv == -INFINITY) continue;
    double d = zv - m;
    double e = exp(d);
    S += e;
    U += d * e;
  }
  double H = log(S) - U / S;
  double s = H / log((double)V);
  if (s < 0.0) s = 0.0;
  if (s > 1.0) s = 1.0;
  return s;
}

int cwlo_score_tokens(const float* logits, int64_t ld, int32_t T, int32_t V, double* score) {
  if (!logits || !score || T < 0 || V < 2 || ld < V) return CWLO_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int32_t t = 0; t < T; ++t) score[t] = entropy_row(logits + (int64_t)t * ld, V);
  return CWLO_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Sec. III-B (a chunk is judged by its mean complexity against thresholds): chunk means are compared in fixed point so that
 * the partition is a function of the fp32 score array alone, independent of summation order.
 * ------------------------------------------------------------------------------------------- */
int64_t cwlo_quantise(float s) {
  if (isnan(s)) return Q24;
  double c = (double)s;
  if (c < 0.0) c = 0.0;
  if (c > 1.0) c = 1.0;
  return (int64_t)floor(c * (double)Q24);
}

static int64_t threshold_q(float theta) { return (int64_t)floor((double)theta * (double)Q24); }

/* Sec. III-C / IV-C rule-based mapping: the rung is the number of thresholds the chunk mean
 * reaches (mean >= theta_k  <=>  sum >= Theta_k * len). */
int32_t cwlo_rung(int64_t sum, int64_t len, const cwlo_policy* p) {
  int32_t k = 0;
  for (int32_t j = 0; j + 1 < p->n_rungs; ++j)
    if (sum >= threshold_q(p->threshold[j]) * len) ++k;
  return k;
}

static int policy_ok(const cwlo_policy* p) {
  if (!p || p->n_rungs < 1 || p->n_rungs > CWLO_MAX_RUNGS) return 0;
  if (p->min_len < 1 || p->max_len < p->min_len) return 0;
  if ((int64_t)p->min_len + (int64_t)p->max_len > (1 << 19)) return 0;
  if (p->window < 0 || p->window > p->min_len) return 0;
  for (int32_t k = 0; k < p->n_rungs; ++k) {
    if (p->rung_rank[k] < 0) return 0;
    if (k > 0 && p->rung_rank[k] < p->rung_rank[k - 1]) return 0;
  }
  for (int32_t k = 0; k + 1 < p->n_rungs; ++k) {
    float th = p->threshold[k];
    if (!(th >= 0.0f && th <= 1.0f)) return 0;
    if (k > 0 && !(th > p->threshold[k - 1])) return 0;
  }
  return 1;
}

int cwlo_partition(const float* score, const int32_t* cu, int32_t n_seq, int32_t T,
                   const cwlo_policy* p, int32_t* offsets, int32_t* rank, float* scale,
                   int32_t* rung, int32_t* flags, int32_t* n_chunks, int32_t capacity) {
  if (!score || !cu || !offsets || !rank || !scale || !rung || !flags || !n_chunks) return CWLO_ERR_ARG;
  if (n_seq < 0 || T < 0 || capacity < 0 || !policy_ok(p)) return CWLO_ERR_ARG;
  if (cu[0] != 0 || cu[n_seq] != T) return CWLO_ERR_ARG;
  for (int32_t n = 0; n < n_seq; ++n)
    if (cu[n + 1] < cu[n]) return CWLO_ERR_ARG;

  /* exclusive prefix sums of the quantised scores */
  int64_t* P = (int64_t*)malloc(sizeof(int64_t) * ((size_t)T + 1));
  if (!P) return CWLO_ERR_ARG;
  P[0] = 0;
  for (int32_t t = 0; t < T; ++t) P[t + 1] = P[t] + cwlo_quantise(score[t]);

  const int32_t Lmin = p->min_len, Lmax = p->max_len, K = p->n_rungs;
  int32_t C = 0;
  int status = CWLO_OK;
  offsets[0] = 0;

  for (int32_t n = 0; n < n_seq && status == CWLO_OK; ++n) {
    const int32_t S = cu[n], E = cu[n + 1];
    const int32_t first_chunk = C;
    /* -- the greedy online walk (Sec. III-B): grow the open chunk one token at a time, close it
     *    at the length cap or where the next L_min tokens fall in another complexity class -- */
    int32_t b = S;
    while (b < E) {
      int32_t e;
      if (E - b < 2 * Lmin) {
        e = E; /* two legal chunks do not fit: take the rest */
      } else {
        e = b + Lmin;
        for (;;) {
          if (e - b >= Lmax) break;
          int32_t open_rung  = cwlo_rung(P[e] - P[b], e - b, p);
          int32_t ahead_rung = cwlo_rung(P[e + Lmin] - P[e], Lmin, p);
          if (open_rung != ahead_rung) break;
          e = e + 1;
          if (E - e < Lmin) { e = E; break; } /* the tail would be too short: absorb it */
        }
      }
      if (C >= capacity) { status = CWLO_ERR_CAPACITY; break; }
      offsets[C + 1] = e;
      flags[C] = (b == S) ? 1 : 0;
      rung[C] = cwlo_rung(P[e] - P[b], e - b, p);
      ++C;
      b = e;
    }
    if (status != CWLO_OK) break;

    /* -- budget on high-capacity regions (Sec. III-B): at most hi_budget chunks of this
     *    sequence stay on the top rung; the ones with the smallest means step down one rung -- */
    if (p->hi_budget >= 0 && K >= 2 && C > first_chunk) {
      /* the ranking is taken over the rungs as the walk left them, before any demotion */
      int32_t* walked = (int32_t*)malloc(sizeof(int32_t) * (size_t)(C - first_chunk));
      for (int32_t c = first_chunk; c < C; ++c) walked[c - first_chunk] = rung[c];
      for (int32_t c = first_chunk; c < C; ++c) {
        if (walked[c - first_chunk] != K - 1) continue;
        int64_t sum_c = P[offsets[c + 1]] - P[offsets[c]], len_c = offsets[c + 1] - offsets[c];
        int32_t better = 0; /* top-rung chunks of this sequence that outrank chunk c */
        for (int32_t d = first_chunk; d < C; ++d) {
          if (d == c || walked[d - first_chunk] != K - 1) continue;
          int64_t sum_d = P[offsets[d + 1]] - P[offsets[d]], len_d = offsets[d + 1] - offsets[d];
          int64_t lhs = sum_d * len_c, rhs = sum_c * len_d; /* mean_d against mean_c */
          if (lhs > rhs || (lhs == rhs && d < c)) ++better;
        }
        if (better >= p->hi_budget) rung[c] = K - 2;
      }
      free(walked);
    }
  }

  if (status == CWLO_OK) {
    for (int32_t c = 0; c < C; ++c) {
      rank[c] = p->rung_rank[rung[c]];
      scale[c] = p->rung_scale[rung[c]];
    }
    *n_chunks = C;
  }
  free(P);
  return status;
}

/* ---------------------------------------------------------------------------------------------
 * Sec. III-D: over a short window after a join the outgoing adapter ramps down linearly while
 * the incoming one ramps up.  The window is the first w rows of the incoming chunk; the ramp
 * takes the w equally spaced values strictly between 0 and 1.
 * ------------------------------------------------------------------------------------------- */
double cwlo_blend_weight(int32_t t, const int32_t* offsets, const int32_t* flags,
                         int32_t n_chunks, int32_t window, int32_t* chunk) {
  int32_t c = 0;
  while (c + 1 < n_chunks && offsets[c + 1] <= t) ++c;
  if (chunk) *chunk = c;
  int32_t j = t - offsets[c];
  if (c == 0 || (flags[c] & 1) || j >= window) return 1.0;
  return (double)(j + 1) / (double)(window + 1);
}

static double bf16_to_double(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* delta[n] = s * sum_{j<r} (sum_k x[k] A[k,j]) B[j,n]   -- one adapter configuration, one row */
static void adapter_row(const uint16_t* x, const uint16_t* A, int64_t lda, const uint16_t* B,
                        int64_t ldb, int32_t d_in, int32_t d_out, int32_t r, double s,
                        double* h, double* delta) {
  for (int32_t n = 0; n < d_out; ++n) delta[n] = 0.0;
  for (int32_t j = 0; j < r; ++j) {
    double acc = 0.0;
    for (int32_t k = 0; k < d_in; ++k) acc += bf16_to_double(x[k]) * bf16_to_double(A[(int64_t)k * lda + j]);
    h[j] = acc;
  }
  for (int32_t j = 0; j < r; ++j)
    for (int32_t n = 0; n < d_out; ++n) delta[n] += h[j] * bf16_to_double(B[(int64_t)j * ldb + n]);
  for (int32_t n = 0; n < d_out; ++n) delta[n] *= s;
}

int cwlo_apply(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
               const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
               int32_t T, int32_t d_in, int32_t d_out, int32_t R,
               const int32_t* offsets, const int32_t* rank, const float* scale,
               const int32_t* flags, int32_t n_chunks, int32_t window,
               const int32_t* rows, int32_t n_rows, double* Y, int64_t ldy) {
  if (!X || !W || !Y || T < 0 || d_in < 1 || d_out < 1 || R < 0 || window < 0) return CWLO_ERR_ARG;
  const int has_adapter = (A != NULL && B != NULL && R > 0);
  if (has_adapter) {
    if (!offsets || !rank || !scale || !flags || n_chunks < 1) return CWLO_ERR_ARG;
    if (offsets[0] != 0 || offsets[n_chunks] != T) return CWLO_ERR_ARG;
    for (int32_t c = 0; c < n_chunks; ++c)
      if (rank[c] < 0 || rank[c] > R || offsets[c + 1] < offsets[c]) return CWLO_ERR_ARG;
  }
  const int32_t count = rows ? n_rows : T;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t i = 0; i < count; ++i) {
    const int32_t t = rows ? rows[i] : i;
    if (t < 0 || t >= T) { bad = 1; continue; }
    const uint16_t* x = X + (int64_t)t * ldx;
    double* y = Y + (int64_t)i * ldy;
    /* base projection x_t W */
    for (int32_t n = 0; n < d_out; ++n) y[n] = 0.0;
    for (int32_t k = 0; k < d_in; ++k) {
      double xk = bf16_to_double(x[k]);
      const uint16_t* w = W + (int64_t)k * ldw;
      for (int32_t n = 0; n < d_out; ++n) y[n] += xk * bf16_to_double(w[n]);
    }
    if (!has_adapter) continue;
    int32_t c;
    double lam = cwlo_blend_weight(t, offsets, flags, n_chunks, window, &c);
    double* h = (double*)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
    double* d_in_c = (double*)malloc(sizeof(double) * (size_t)d_out);
    double* d_out_p = (double*)malloc(sizeof(double) * (size_t)d_out);
    /* incoming (own chunk) adapter output */
    adapter_row(x, A, lda, B, ldb, d_in, d_out, rank[c], (double)scale[c], h, d_in_c);
    if (lam < 1.0) {
      /* outgoing (previous chunk) adapter output, then the literal cross-fade */
      adapter_row(x, A, lda, B, ldb, d_in, d_out, rank[c - 1], (double)scale[c - 1], h, d_out_p);
      for (int32_t n = 0; n < d_out; ++n) y[n] += (1.0 - lam) * d_out_p[n] + lam * d_in_c[n];
    } else {
      for (int32_t n = 0; n < d_out; ++n) y[n] += d_in_c[n];
    }
    free(h); free(d_in_c); free(d_out_p);
  }
  return bad ? CWLO_ERR_ARG : CWLO_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Sec. III-G / IV-F, batch alignment: sequences of a batch are bucketed by complexity percentile so that the
 * chunk joins of a bucket line up, while every sequence keeps its own rank choices.  The paper gives one
 * sentence; this build's reading, step by step:
 *   1. the complexity of a sequence is the mean of its quantised scores (sum_n / len_n, compared exactly by
 *      cross-multiplication); sequences are ordered by it, ascending, the lower index first on ties, empty
 *      sequences before all others;
 *   2. the sequence at position i of that order (0-based) falls into bucket floor(i * n_buckets / n_seq):
 *      percentile bands of (almost) equal population;
 *   3. per bucket the scores are pooled position by position (positions count from each sequence's start):
 *      S[j] = sum of q over the members that have a token at position j, N[j] = how many do;
 *   4. the greedy walk of Sec. III-B (cwlo_partition's rule) runs ONCE per bucket on the pooled track over
 *      positions [0, longest member): the mean of a span is sum S / sum N, i.e. the mean over all member
 *      tokens at those positions; its cuts are the bucket's shared joins;
 *   5. a member takes every shared join that leaves it at least L_min tokens (join <= len_n - L_min), so
 *      its last chunk absorbs what a later join would have cut off too short;
 *   6. rung, budget, rank and scale of each chunk come from the sequence's OWN scores, as in cwlo_partition.
 * Outputs: the chunk table in sequence order, bucket[n] and order_pos[n] (position of sequence n in the
 * complexity order).
 * ------------------------------------------------------------------------------------------- */
static int32_t pooled_rung(int64_t sum, int64_t count, const cwlo_policy* p) {
  int32_t k = 0;
  for (int32_t j = 0; j + 1 < p->n_rungs; ++j)
    if (sum >= threshold_q(p->threshold[j]) * count) ++k;
  return k;
}

int cwlo_batch_align(const float* score, const int32_t* cu, int32_t n_seq, int32_t T,
                     const cwlo_policy* p, int32_t n_buckets,
                     int32_t* offsets, int32_t* rank, float* scale, int32_t* rung, int32_t* flags,
                     int32_t* n_chunks, int32_t capacity, int32_t* bucket, int32_t* order_pos) {
  if (!score || !cu || !offsets || !rank || !scale || !rung || !flags || !n_chunks || !bucket || !order_pos)
    return CWLO_ERR_ARG;
  if (n_seq < 0 || T < 0 || capacity < 0 || n_buckets < 1 || !policy_ok(p)) return CWLO_ERR_ARG;
  if (cu[0] != 0 || cu[n_seq] != T) return CWLO_ERR_ARG;
  for (int32_t n = 0; n < n_seq; ++n)
    if (cu[n + 1] < cu[n]) return CWLO_ERR_ARG;
  const int32_t Lmin = p->min_len, Lmax = p->max_len, K = p->n_rungs;

  int64_t* P = (int64_t*)malloc(sizeof(int64_t) * ((size_t)T + 1));      /* prefix sums of the packed scores */
  int64_t* PS = (int64_t*)malloc(sizeof(int64_t) * ((size_t)T + 2));     /* pooled track of one bucket, prefix sums */
  int64_t* PN = (int64_t*)malloc(sizeof(int64_t) * ((size_t)T + 2));
  int32_t* joins = (int32_t*)malloc(sizeof(int32_t) * ((size_t)T + 2));
  P[0] = 0;
  for (int32_t t = 0; t < T; ++t) P[t + 1] = P[t] + cwlo_quantise(score[t]);

  /* 1./2. complexity order and percentile buckets */
  for (int32_t n = 0; n < n_seq; ++n) {
    const int64_t sum_n = P[cu[n + 1]] - P[cu[n]], len_n = cu[n + 1] - cu[n];
    int32_t before = 0;
    for (int32_t m = 0; m < n_seq; ++m) {
      if (m == n) continue;
      const int64_t sum_m = P[cu[m + 1]] - P[cu[m]], len_m = cu[m + 1] - cu[m];
      int m_first;
      if (len_m == 0 || len_n == 0) {
        if (len_m == 0 && len_n == 0) m_first = m < n;
        else m_first = (len_m == 0);
      } else {
        const int64_t lhs = sum_m * len_n, rhs = sum_n * len_m;          /* mean_m against mean_n */
        m_first = lhs < rhs || (lhs == rhs && m < n);
      }
      if (m_first) ++before;
    }
    order_pos[n] = before;
    bucket[n] = (int32_t)(((int64_t)before * n_buckets) / n_seq);
  }

  int32_t C = 0;
  int status = CWLO_OK;
  offsets[0] = 0;
  /* chunks are emitted in sequence order; the shared joins of a sequence's bucket are worked out when needed */
  for (int32_t n = 0; n < n_seq && status == CWLO_OK; ++n) {
    const int32_t S = cu[n], len_n = cu[n + 1] - cu[n], k = bucket[n];
    if (len_n == 0) continue;
    /* 3. pooled track of bucket k */
    int32_t L = 0;
    for (int32_t m = 0; m < n_seq; ++m)
      if (bucket[m] == k && cu[m + 1] - cu[m] > L) L = cu[m + 1] - cu[m];
    PS[0] = 0; PN[0] = 0;
    for (int32_t j = 0; j < L; ++j) {
      int64_t s = 0, c = 0;
      for (int32_t m = 0; m < n_seq; ++m)
        if (bucket[m] == k && cu[m + 1] - cu[m] > j) { s += cwlo_quantise(score[cu[m] + j]); c += 1; }
      PS[j + 1] = PS[j] + s; PN[j + 1] = PN[j] + c;
    }
    /* 4. the walk of Sec. III-B on the pooled track over [0, L) */
    int32_t n_joins = 0;
    int32_t b = 0;
    while (b < L) {
      int32_t e;
      if (L - b < 2 * Lmin) {
        e = L;
      } else {
        e = b + Lmin;
        for (;;) {
          if (e - b >= Lmax) break;
          int32_t open_rung  = pooled_rung(PS[e] - PS[b], PN[e] - PN[b], p);
          int32_t ahead_rung = pooled_rung(PS[e + Lmin] - PS[e], PN[e + Lmin] - PN[e], p);
          if (open_rung != ahead_rung) break;
          e = e + 1;
          if (L - e < Lmin) { e = L; break; }
        }
      }
      if (e < L) joins[n_joins++] = e;
      b = e;
    }
    /* 5. the member's own chunks */
    const int32_t first_chunk = C;
    int32_t start = 0;
    for (int32_t i = 0; i <= n_joins && status == CWLO_OK; ++i) {
      int32_t end;
      if (i < n_joins && joins[i] <= len_n - Lmin) end = joins[i];
      else end = len_n;
      if (C >= capacity) { status = CWLO_ERR_CAPACITY; break; }
      offsets[C + 1] = S + end;
      flags[C] = (start == 0) ? 1 : 0;
      rung[C] = cwlo_rung(P[S + end] - P[S + start], end - start, p);     /* 6. own scores */
      ++C;
      start = end;
      if (end == len_n) break;
    }
    if (status != CWLO_OK) break;
    /* 6. budget on top-rung chunks, per sequence, exactly as in cwlo_partition */
    if (p->hi_budget >= 0 && K >= 2 && C > first_chunk) {
      int32_t* walked = (int32_t*)malloc(sizeof(int32_t) * (size_t)(C - first_chunk));
      for (int32_t c = first_chunk; c < C; ++c) walked[c - first_chunk] = rung[c];
      for (int32_t c = first_chunk; c < C; ++c) {
        if (walked[c - first_chunk] != K - 1) continue;
        int64_t sum_c = P[offsets[c + 1]] - P[offsets[c]], len_c = offsets[c + 1] - offsets[c];
        int32_t better = 0;
        for (int32_t d = first_chunk; d < C; ++d) {
          if (d == c || walked[d - first_chunk] != K - 1) continue;
          int64_t sum_d = P[offsets[d + 1]] - P[offsets[d]], len_d = offsets[d + 1] - offsets[d];
          int64_t lhs = sum_d * len_c, rhs = sum_c * len_d;
          if (lhs > rhs || (lhs == rhs && d < c)) ++better;
        }
        if (better >= p->hi_budget) rung[c] = K - 2;
      }
      free(walked);
    }
  }
  if (status == CWLO_OK) {
    for (int32_t c = 0; c < C; ++c) {
      rank[c] = p->rung_rank[rung[c]];
      scale[c] = p->rung_scale[rung[c]];
    }
    *n_chunks = C;
  }
  free(P); free(PS); free(PN); free(joins);
  return status;
}

/* ---------------------------------------------------------------------------------------------
 * Sec. III-D, centred placement of the cross-fade window (a variant: the paper says only that the
 * window is short).  The w rows AROUND a join are blended: the last floor(w/2) rows of the outgoing
 * chunk and the first ceil(w/2) rows of the incoming chunk.  Counted from the window's first row,
 * row i = 0..w-1 gets the weight (i+1)/(w+1) for the incoming configuration, as in the causal
 * placement.  A join into the first chunk of a sequence has no window.  Where a chunk is so short
 * that the window after its opening join and the one before its closing join meet, the rows of the
 * opening join's window win.
 *   returns lam, the weight of configuration *cfg_in; *cfg_out carries 1 - lam (equal to *cfg_in
 *   and lam = 1 outside every window).
 * ------------------------------------------------------------------------------------------- */
double cwlo_blend_weight_centred(int32_t t, const int32_t* offsets, const int32_t* flags,
                                 int32_t n_chunks, int32_t window, int32_t* cfg_in, int32_t* cfg_out) {
  int32_t c = 0;
  while (c + 1 < n_chunks && offsets[c + 1] <= t) ++c;
  const int32_t before = window / 2;          /* rows of the window in the outgoing chunk */
  const int32_t after = window - before;      /* rows of the window in the incoming chunk */
  const int32_t j = t - offsets[c];
  const int32_t len = offsets[c + 1] - offsets[c];
  int32_t in = c, out = c;
  double lam = 1.0;
  if (c > 0 && !(flags[c] & 1) && j < after) {
    /* head of the incoming chunk: window row i = before + j */
    lam = (double)(before + j + 1) / (double)(window + 1);
    in = c; out = c - 1;
  } else if (c + 1 < n_chunks && !(flags[c + 1] & 1) && len - j <= before) {
    /* tail of the outgoing chunk: the window starts `before` rows ahead of the join */
    lam = (double)(before - (len - j) + 1) / (double)(window + 1);
    in = c + 1; out = c;
  }
  if (cfg_in) *cfg_in = in;
  if (cfg_out) *cfg_out = out;
  return lam;
}

/* Adapted projection with the centred window: for a row whose window joins configurations `out` and `in`,
 *   y_t = x_t W + (1-lam_t) s_out (x_t A[:, :r_out]) B[:r_out, :] + lam_t s_in (x_t A[:, :r_in]) B[:r_in, :],
 * the three products computed one by one and then combined.  Arguments as cwlo_apply. */
int cwlo_apply_centred(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                       const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                       int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                       const int32_t* offsets, const int32_t* rank, const float* scale,
                       const int32_t* flags, int32_t n_chunks, int32_t window,
                       const int32_t* rows, int32_t n_rows, double* Y, int64_t ldy) {
  if (!X || !W || !Y || T < 0 || d_in < 1 || d_out < 1 || R < 0 || window < 0) return CWLO_ERR_ARG;
  const int has_adapter = (A != NULL && B != NULL && R > 0);
  if (has_adapter) {
    if (!offsets || !rank || !scale || !flags || n_chunks < 1) return CWLO_ERR_ARG;
    if (offsets[0] != 0 || offsets[n_chunks] != T) return CWLO_ERR_ARG;
    for (int32_t c = 0; c < n_chunks; ++c)
      if (rank[c] < 0 || rank[c] > R || offsets[c + 1] < offsets[c]) return CWLO_ERR_ARG;
  }
  const int32_t count = rows ? n_rows : T;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t i = 0; i < count; ++i) {
    const int32_t t = rows ? rows[i] : i;
    if (t < 0 || t >= T) { bad = 1; continue; }
    const uint16_t* x = X + (int64_t)t * ldx;
    double* y = Y + (int64_t)i * ldy;
    for (int32_t n = 0; n < d_out; ++n) y[n] = 0.0;
    for (int32_t k = 0; k < d_in; ++k) {
      double xk = bf16_to_double(x[k]);
      const uint16_t* w = W + (int64_t)k * ldw;
      for (int32_t n = 0; n < d_out; ++n) y[n] += xk * bf16_to_double(w[n]);
    }
    if (!has_adapter) continue;
    int32_t in, out;
    double lam = cwlo_blend_weight_centred(t, offsets, flags, n_chunks, window, &in, &out);
    double* h = (double*)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
    double* d_new = (double*)malloc(sizeof(double) * (size_t)d_out);
    double* d_old = (double*)malloc(sizeof(double) * (size_t)d_out);
    adapter_row(x, A, lda, B, ldb, d_in, d_out, rank[in], (double)scale[in], h, d_new);
    if (lam < 1.0) {
      adapter_row(x, A, lda, B, ldb, d_in, d_out, rank[out], (double)scale[out], h, d_old);
      for (int32_t n = 0; n < d_out; ++n) y[n] += (1.0 - lam) * d_old[n] + lam * d_new[n];
    } else {
      for (int32_t n = 0; n < d_out; ++n) y[n] += d_new[n];
    }
    free(h); free(d_new); free(d_old);
  }
  return bad ? CWLO_ERR_ARG : CWLO_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Decode-time scheduler (Sec. III-A, III-B, III-F: scores arrive as tokens stream in, tokens are
 * grouped as they arrive, and the scheduler keeps its state from step to step).  The paper names the constraints only; the rule is
 * this build's causal reading: a token may open a new chunk only on what has been seen so far.
 *
 * Per sequence: the open chunk's length and the rung it was opened on (a chunk's configuration is
 * fixed while it is open), the previous chunk's rung, and the quantised scores of the last L_min
 * tokens.  On a new token with quantised score q:
 *   1. q enters the trailing window (the last min(L_min, tokens seen) scores, the new one included);
 *   2. the first token of a sequence opens the first chunk on the rung of that window;
 *   3. otherwise, if the open chunk holds at least L_min tokens and either holds L_max of them or
 *      the window's rung differs from the open chunk's rung, the token opens a new chunk on the
 *      window's rung (with a budget H, a chunk that would open on the top rung after H such
 *      chunks opens one rung lower);
 *   4. the token is row j of its chunk; rows j < w of a chunk that is not the first of its
 *      sequence are cross-faded with lambda = (j+1)/(w+1) (Sec. III-D), all others have lambda = 1.
 * ------------------------------------------------------------------------------------------- */
int cwlo_stream_reset(cwlo_stream_state* st) {
  if (!st) return CWLO_ERR_ARG;
  st->pos = 0; st->len = 0; st->cur_rung = 0; st->prev_rung = -1; st->hi_used = 0; st->first = 1;
  for (int i = 0; i < CWLO_STREAM_MAX_MIN_LEN; ++i) st->ring[i] = 0;
  return CWLO_OK;
}

int cwlo_stream_step(cwlo_stream_state* st, float score, const cwlo_policy* p, cwlo_row_gate* out) {
  if (!st || !out || !policy_ok(p) || p->min_len > CWLO_STREAM_MAX_MIN_LEN) return CWLO_ERR_ARG;
  const int32_t L = p->min_len;
  /* 1. trailing window */
  st->ring[st->pos % L] = cwlo_quantise(score);
  const int32_t n_win = (st->pos + 1 < L) ? st->pos + 1 : L;
  int64_t win = 0;
  for (int32_t i = 0; i < n_win; ++i) win += st->ring[i];     /* slots 0..n_win-1 hold exactly the last n_win scores */
  int32_t r_win = cwlo_rung(win, n_win, p);
  /* 2./3. open a chunk? */
  int open = 0;
  if (st->pos == 0) { open = 1; st->first = 1; }
  else if (st->len >= L && (st->len >= p->max_len || r_win != st->cur_rung)) { open = 1; st->first = 0; }
  if (open) {
    if (p->hi_budget >= 0 && p->n_rungs >= 2 && r_win == p->n_rungs - 1) {
      if (st->hi_used >= p->hi_budget) r_win = p->n_rungs - 2; else st->hi_used += 1;
    }
    st->prev_rung = (st->pos == 0) ? -1 : st->cur_rung;
    st->cur_rung = r_win;
    st->len = 0;
  }
  /* 4. this token's row descriptor */
  const int32_t j = st->len;
  st->len += 1;
  st->pos += 1;
  out->pos_in_chunk = j;
  out->opened = open;
  out->rank_in = p->rung_rank[st->cur_rung];
  out->scale_in = p->rung_scale[st->cur_rung];
  out->rank_out = 0; out->scale_out = 0.0f; out->lambda = 1.0f;
  if (!st->first && j < p->window) {
    out->lambda = (float)(j + 1) / (float)(p->window + 1);
    out->rank_out = p->rung_rank[st->prev_rung];
    out->scale_out = p->rung_scale[st->prev_rung];
  }
  return CWLO_OK;
}

/* Adapted projection with one descriptor per row (decode: every row is another sequence's newest token):
 *   y_t = x_t W + (1-lam_t) s_out (x_t A[:, :r_out]) B[:r_out, :] + lam_t s_in (x_t A[:, :r_in]) B[:r_in, :]  */
int cwlo_apply_rows(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                    const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                    int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                    const cwlo_row_gate* gates, double* Y, int64_t ldy) {
  if (!X || !W || !A || !B || !gates || !Y || T < 0 || d_in < 1 || d_out < 1 || R < 1) return CWLO_ERR_ARG;
  for (int32_t t = 0; t < T; ++t)
    if (gates[t].rank_in < 0 || gates[t].rank_in > R || gates[t].rank_out < 0 || gates[t].rank_out > R) return CWLO_ERR_ARG;
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t t = 0; t < T; ++t) {
    const uint16_t* x = X + (int64_t)t * ldx;
    double* y = Y + (int64_t)t * ldy;
    for (int32_t n = 0; n < d_out; ++n) y[n] = 0.0;
    for (int32_t k = 0; k < d_in; ++k) {
      double xk = bf16_to_double(x[k]);
      const uint16_t* w = W + (int64_t)k * ldw;
      for (int32_t n = 0; n < d_out; ++n) y[n] += xk * bf16_to_double(w[n]);
    }
    double* h = (double*)malloc(sizeof(double) * (size_t)R);
    double* d_new = (double*)malloc(sizeof(double) * (size_t)d_out);
    double* d_old = (double*)malloc(sizeof(double) * (size_t)d_out);
    const double lam = (double)gates[t].lambda;
    adapter_row(x, A, lda, B, ldb, d_in, d_out, gates[t].rank_in, (double)gates[t].scale_in, h, d_new);
    if (lam < 1.0) {
      adapter_row(x, A, lda, B, ldb, d_in, d_out, gates[t].rank_out, (double)gates[t].scale_out, h, d_old);
      for (int32_t n = 0; n < d_out; ++n) y[n] += (1.0 - lam) * d_old[n] + lam * d_new[n];
    } else {
      for (int32_t n = 0; n < d_out; ++n) y[n] += d_new[n];
    }
    free(h); free(d_new); free(d_old);
  }
  return CWLO_OK;
}

/* ---------------------------------------------------------------------------------------------
 * Token complexity estimator with the further signals of Sec. III-A: (i) next-token entropy,
 * (ii) n-gram novelty against the recent context, (iv) a positional prior that favours early
 * steps.  The paper lists the signals and gives no formula; this build's reading:
 *   e_t   normalised entropy of the token's logit row (as cwlo_score_tokens)
 *   nu_t  1 if the n-gram ending at t (token ids x[t-n+1..t]) ends at none of the previous
 *         `context` positions of the same sequence, else 0; the first n-1 tokens of a sequence,
 *         which have no complete n-gram yet, count as novel
 *   pi_t  max(0, 1 - p / prior_span), p = position of t inside its sequence
 *   score = clamp(w_e e_t + w_n nu_t + w_p pi_t, 0, 1)      (a NaN entropy stays NaN)
 * ------------------------------------------------------------------------------------------- */
int cwlo_score_tokens_mixed(const float* logits, int64_t ld, int32_t T, int32_t V,
                            const int32_t* token_ids, const int32_t* cu, int32_t n_seq,
                            const cwlo_signal_mix* mix, double* score) {
  if (!logits || !token_ids || !cu || !mix || !score || T < 0 || V < 2 || ld < V || n_seq < 0) return CWLO_ERR_ARG;
  if (mix->ngram < 1 || mix->ngram > 8 || mix->context < 1 || mix->prior_span < 1) return CWLO_ERR_ARG;
  if (!(mix->w_entropy >= 0.f) || !(mix->w_novelty >= 0.f) || !(mix->w_prior >= 0.f)) return CWLO_ERR_ARG;
  if (cu[0] != 0 || cu[n_seq] != T) return CWLO_ERR_ARG;
  for (int32_t s = 0; s < n_seq; ++s) {
    if (cu[s + 1] < cu[s]) return CWLO_ERR_ARG;
    for (int32_t t = cu[s]; t < cu[s + 1]; ++t) {
      const int32_t p = t - cu[s];
      const double e = entropy_row(logits + (int64_t)t * ld, V);
      double nu = 1.0;
      if (p >= mix->ngram - 1) {
        int32_t lo = t - mix->context;
        if (lo < cu[s] + mix->ngram - 1) lo = cu[s] + mix->ngram - 1;
        for (int32_t u = lo; u < t && nu == 1.0; ++u) {
          int same = 1;
          for (int32_t i = 0; i < mix->ngram; ++i)
            if (token_ids[u - i] != token_ids[t - i]) { same = 0; break; }
          if (same) nu = 0.0;
        }
      }
      double pi = 1.0 - (double)p / (double)mix->prior_span;
      if (pi < 0.0) pi = 0.0;
      double v = (double)mix->w_entropy * e + (double)mix->w_novelty * nu + (double)mix->w_prior * pi;
      if (!isnan(v)) { if (v < 0.0) v = 0.0; if (v > 1.0) v = 1.0; }
      score[t] = v;
    }
  }
  return CWLO_OK;
}
