/*
 * cwlo.h -- fp64 CPU oracle for the ChunkWise-LoRA hot path (TEST INFRASTRUCTURE ONLY).
 *
 * This is a plain, slow, single-translation-unit restatement of what the method computes,
 * written from the paper's prose (it prints no equations): the token complexity estimator's
 * entropy signal (Sec. III-A (i), Sec. IV-A), the adaptive chunker (Sec. III-B, IV-B), the
 * per-chunk rank & scale selector on a prefix-slice rank ladder (Sec. III-C, IV-C), the
 * boundary-safe linear cross-fade (Sec. III-D) and the adapted projection on the LoRA-carrying
 * projections (Sec. III-F, IV-E).
 *
 * It shares no code, header, table or helper with the CUDA library and must never be linked
 * or imported by it.  Only the test-suite, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  All pointers are HOST pointers.  Floating-point results are fp64.
 *
 * Pin status (see tests/test_oracle_*.py):
 *   score     pinned  (closed forms, invariances, binary-entropy special case, library log-softmax)
 *   rung      pinned  (exhaustive tiny ranges, length-1 reduction, monotonicity)
 *   chunker   parity unpinned against the paper (it prints neither a rule nor a worked example);
 *             pinned internally by hand-traced cases, invariants and an independent brute force
 *   budget    pinned  (definition: keep the H largest means, earlier index wins ties)
 *   blend     pinned  (weights sum to one, equal spacing, convex combination of single-chunk runs)
 *   apply     pinned  (merged-weight LoRA, r = 0 base, hand-expanded tiny case, linearity)
 *   align     parity unpinned against the paper (one sentence, no rule); pinned internally: one bucket per sequence
 *             reduces to the pinned cwlo_partition, a hand-traced pooled walk, invariants, an exact-rational brute force
 *   centred   pinned  (window sums, equal spacing, the causal ramp shifted, convex combination of single-
 *             configuration runs, hand-expanded tiny case)
 *   mixed     pinned  (weights (1,0,0) = entropy score, hand-traced novelty, closed-form prior, set-based brute force)
 *   stream    parity unpinned against the paper (no rule printed); pinned internally by hand-traced runs,
 *             invariants and an independent brute force; apply_rows pinned against cwlo_apply on equivalent tables
 */
#ifndef CWLO_H
#define CWLO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CWLO_MAX_RUNGS 8

/* Policy of the chunker and the selector.  Field meaning:
 *   rung_rank[k]   prefix rank of ladder rung k (non-decreasing in k)
 *   rung_scale[k]  gating scale of rung k (the harness passes alpha / rank)
 *   threshold[k]   mean score at or above which a chunk climbs from rung k to rung k+1
 *   min_len/max_len  the chunker's length bounds (L_min, L_max)
 *   window         cross-fade window length w in tokens (0 <= w <= L_min)
 *   hi_budget      maximum number of top-rung chunks per sequence; negative = unlimited */
typedef struct {
  int32_t n_rungs;
  int32_t rung_rank[CWLO_MAX_RUNGS];
  float   rung_scale[CWLO_MAX_RUNGS];
  float   threshold[CWLO_MAX_RUNGS - 1];
  int32_t min_len, max_len;
  int32_t window;
  int32_t hi_budget;
} cwlo_policy;

/* return codes */
enum { CWLO_OK = 0, CWLO_ERR_ARG = 1, CWLO_ERR_CAPACITY = 4 };

/* Normalised next-token entropy of each logit row, in [0,1] (Sec. III-A signal (i)).
 * logits: [T, V] fp32, row stride ld (elements).  score: [T] fp64. */
int cwlo_score_tokens(const float* logits, int64_t ld, int32_t T, int32_t V, double* score);

/* Fixed-point image of a score: floor(clamp(s,0,1) * 2^24); NaN maps to 2^24. */
int64_t cwlo_quantise(float s);

/* Ladder rung of the span whose quantised scores sum to `sum` over `len` tokens. */
int32_t cwlo_rung(int64_t sum, int64_t len, const cwlo_policy* p);

/* Adaptive chunker + rank/scale selector (Sec. III-B, III-C).
 * score [T] fp32; cu_seqlens [n_seq+1] (cu[0]=0, cu[n_seq]=T, non-decreasing).
 * Outputs (capacity entries, offsets capacity+1): chunk offsets, rank, scale, rung,
 * flags (bit0 = first chunk of its sequence), *n_chunks. */
int cwlo_partition(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                   const cwlo_policy* p, int32_t* offsets, int32_t* rank, float* scale,
                   int32_t* rung, int32_t* flags, int32_t* n_chunks, int32_t capacity);

/* Cross-fade weight of the incoming configuration for row `t` (Sec. III-D):
 * rows j = 0..w-1 of a chunk that is not first of its sequence get (j+1)/(w+1), others 1.
 * *chunk receives the index of the chunk holding row t. */
double cwlo_blend_weight(int32_t t, const int32_t* offsets, const int32_t* flags,
                         int32_t n_chunks, int32_t window, int32_t* chunk);

/* Adapted projection (Sec. III-F with the cross-fade of Sec. III-D):
 *   y_t = x_t W + (1-lam_t) s_p (x_t A[:, :r_p]) B[:r_p, :] + lam_t s_c (x_t A[:, :r_c]) B[:r_c, :]
 * X [T,d_in], W [d_in,d_out], A [d_in,R], B [R,d_out] are bf16 bit patterns (uint16), row-major
 * with explicit leading dimensions; A == NULL or B == NULL or R == 0 means no adapter.
 * rows == NULL computes every row into Y [T,d_out]; otherwise rows[0..n_rows) are computed and
 * written to Y [n_rows, d_out] in list order (row-subset mode).  Y is fp64, row stride ldy. */
int cwlo_apply(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
               const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
               int32_t T, int32_t d_in, int32_t d_out, int32_t R,
               const int32_t* offsets, const int32_t* rank, const float* scale,
               const int32_t* flags, int32_t n_chunks, int32_t window,
               const int32_t* rows, int32_t n_rows, double* Y, int64_t ldy);

/* Batch alignment (Sec. III-G, IV-F): sequences are bucketed by complexity percentile and the members of a
 * bucket share their chunk joins (worked out on the bucket's pooled score track), while rung, budget, rank
 * and scale stay per sequence.  See cwlo.c for the steps.  Table outputs as cwlo_partition;
 * bucket[n_seq] and order_pos[n_seq] receive each sequence's bucket and its position in the complexity order. */
int cwlo_batch_align(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                     const cwlo_policy* p, int32_t n_buckets,
                     int32_t* offsets, int32_t* rank, float* scale, int32_t* rung, int32_t* flags,
                     int32_t* n_chunks, int32_t capacity, int32_t* bucket, int32_t* order_pos);

/* The cross-fade window placed AROUND the join instead of after it (Sec. III-D variant): the last
 * floor(w/2) rows of the outgoing chunk and the first ceil(w/2) rows of the incoming chunk; window
 * row i gets (i+1)/(w+1) for the incoming configuration.  Returns that weight; *cfg_in / *cfg_out
 * receive the chunk indices whose (rank, scale) carry lam and 1 - lam. */
double cwlo_blend_weight_centred(int32_t t, const int32_t* offsets, const int32_t* flags,
                                 int32_t n_chunks, int32_t window, int32_t* cfg_in, int32_t* cfg_out);
int cwlo_apply_centred(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                       const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                       int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                       const int32_t* offsets, const int32_t* rank, const float* scale,
                       const int32_t* flags, int32_t n_chunks, int32_t window,
                       const int32_t* rows, int32_t n_rows, double* Y, int64_t ldy);

/* Mix of complexity signals (Sec. III-A (i), (ii), (iv)); see cwlo.c for the definitions. */
typedef struct {
  float   w_entropy, w_novelty, w_prior;   /* non-negative weights */
  int32_t ngram;                           /* n of the n-gram, 1..8 */
  int32_t context;                         /* previous positions searched, >= 1 */
  int32_t prior_span;                      /* positions over which the prior falls from 1 to 0, >= 1 */
} cwlo_signal_mix;
int cwlo_score_tokens_mixed(const float* logits, int64_t ld, int32_t T, int32_t V,
                            const int32_t* token_ids, const int32_t* cu_seqlens, int32_t n_seq,
                            const cwlo_signal_mix* mix, double* score);

/* Decode-time scheduler state of ONE sequence and the descriptor of one row (see cwlo.c for the rule). */
#define CWLO_STREAM_MAX_MIN_LEN 64
typedef struct {
  int32_t pos;        /* tokens seen */
  int32_t len;        /* tokens in the open chunk */
  int32_t cur_rung;   /* rung the open chunk was opened on */
  int32_t prev_rung;  /* rung of the chunk before it (-1: none) */
  int32_t hi_used;    /* top-rung chunks opened so far */
  int32_t first;      /* the open chunk is the first of its sequence */
  int64_t ring[CWLO_STREAM_MAX_MIN_LEN];  /* quantised scores of the last min_len tokens, slot = position mod min_len */
} cwlo_stream_state;
typedef struct {
  int32_t rank_in, rank_out;      /* prefix ranks of the row's own chunk and of the chunk before it */
  float   scale_in, scale_out;    /* their gating scales */
  float   lambda;                 /* cross-fade weight of the own chunk, fp32 (j+1)/(w+1); 1 outside a window */
  int32_t pos_in_chunk;           /* j */
  int32_t opened;                 /* 1 if this token opened a chunk */
} cwlo_row_gate;
int cwlo_stream_reset(cwlo_stream_state* st);
int cwlo_stream_step(cwlo_stream_state* st, float score, const cwlo_policy* p, cwlo_row_gate* out);
int cwlo_apply_rows(const uint16_t* X, int64_t ldx, const uint16_t* W, int64_t ldw,
                    const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb,
                    int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                    const cwlo_row_gate* gates, double* Y, int64_t ldy);

/* Number of threads the row loops of cwlo_score_tokens / cwlo_apply run on (OpenMP). */
int  cwlo_get_threads(void);
void cwlo_set_threads(int n);

#ifdef __cplusplus
}
#endif
#endif
