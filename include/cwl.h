/*
 * cwl.h -- C ABI of the B200 (sm_100a) ChunkWise-LoRA hot path.
 *
 * Three calls follow the paper's pipeline (Sec. III):
 *   cwl_score_tokens  token complexity estimator, entropy signal        (Sec. III-A (i), IV-A)
 *   cwl_partition     adaptive chunker + per-chunk rank/scale selector  (Sec. III-B, III-C, IV-B, IV-C)
 *   cwl_apply         adapted projection with the boundary cross-fade   (Sec. III-D, III-F, IV-E)
 *
 * Conventions for every call
 *   - Pointers marked DEV are device pointers owned by the caller; the library never frees or
 *     keeps them.  Pointers marked HOST are read during the call only.
 *   - All matrices are row-major with an explicit leading dimension in ELEMENTS.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it and the call returns without synchronising.
 *   - Argument errors are reported synchronously through the return value and nothing is
 *     launched.  Problems only visible on the device (chunk table capacity exceeded, a bounded
 *     wait that ran out) are OR-ed as (1 << status) into *status_word (DEV int32, may be NULL);
 *     the caller zeroes it.  The library never traps, prints or exits.
 *   - Calls on distinct streams may run concurrently as long as they use distinct workspaces.
 *   - The library allocates no device memory in these calls; scratch comes from `workspace`,
 *     whose contents never have to be initialised or cleared by the caller.
 *   - Kernels are launched so that their set-up may overlap the end of the kernel ahead of them
 *     in the stream; each waits for that kernel to complete before it reads or writes global
 *     memory, so stream order holds for every buffer.  Launches recorded by a stream capture use
 *     plain stream order.
 */
#ifndef CWL_H
#define CWL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CWL_OK = 0,
  CWL_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, malformed policy */
  CWL_ERR_SHAPE = 2,       /* leading dimension smaller than the row, misaligned pointer or stride */
  CWL_ERR_UNSUPPORTED = 3, /* shape outside the supported set (see each call) */
  CWL_ERR_CAPACITY = 4,    /* chunk table too small (device-side, via status_word) */
  CWL_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than *_workspace_bytes() */
  CWL_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed */
  CWL_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out (device-side, via status_word) */
} cwl_status;

#define CWL_MAX_RUNGS 8
#define CWL_MAX_RANK 256

/* Chunker and selector policy (HOST, copied at call time).  The paper names these knobs
 * (length bounds, average-complexity threshold, budget of high-capacity regions: Sec. III-B;
 * rank ladder and gating scale: Sec. III-C) without giving values. */
typedef struct {
  int32_t n_rungs;                      /* K, 1..CWL_MAX_RUNGS */
  int32_t rung_rank[CWL_MAX_RUNGS];     /* prefix rank of each rung, non-decreasing, >= 0 */
  float   rung_scale[CWL_MAX_RUNGS];    /* gating scale of each rung (e.g. alpha / rank) */
  float   threshold[CWL_MAX_RUNGS - 1]; /* strictly increasing, in [0,1]: mean >= threshold[k] climbs to rung k+1 */
  int32_t min_len, max_len;             /* 1 <= min_len <= max_len, min_len + max_len <= 2^19 */
  int32_t window;                       /* cross-fade window, 0 <= window <= min_len */
  int32_t hi_budget;                    /* max top-rung chunks per sequence; < 0 = unlimited */
} cwl_policy;

/* Chunk table: struct of DEV arrays with `capacity` entries (`offsets` has capacity + 1).
 * Chunk c covers rows [offsets[c], offsets[c+1]); offsets[0] = 0, offsets[n_chunks] = T. */
typedef struct {
  int32_t* offsets;  /* DEV int32 [capacity + 1] */
  int32_t* rank;     /* DEV int32 [capacity]  prefix rank r_c */
  float*   scale;    /* DEV fp32  [capacity]  gating scale s_c */
  int32_t* rung;     /* DEV int32 [capacity]  ladder index (written by cwl_partition, unused by cwl_apply) */
  int32_t* flags;    /* DEV int32 [capacity]  bit0 = first chunk of its sequence (never blended in) */
  int32_t* n_chunks; /* DEV int32 [1] */
  int32_t  capacity;
} cwl_chunk_table;

const char* cwl_status_string(cwl_status s);
int         cwl_version(void);

/* Token complexity score (Sec. III-A signal (i)): normalised entropy of softmax(logits[t, :]),
 *   score[t] = (ln S - U / S) / ln V,  S = sum exp(z - max z),  U = sum (z - max z) exp(z - max z),
 * clamped to [0,1].  -inf logits contribute nothing; a row with NaN or +inf, or of -inf only,
 * scores NaN.  fp32 arithmetic.
 *   logits DEV fp32 [T, V], row stride ld_logits >= V;  score DEV fp32 [T].
 * Errors: INVALID_ARG (NULL, T < 0, V < 2), SHAPE (ld_logits < V).  T == 0 is a no-op. */
cwl_status cwl_score_tokens(const float* logits, int64_t ld_logits, int32_t T, int32_t V,
                            float* score, void* stream);

/* The estimator with the further signals of Sec. III-A mixed in (the paper lists them without formulas):
 *   e_t   the entropy score above
 *   nu_t  n-gram novelty: 1 if the n-gram of token ids ending at t ends at none of the previous `context`
 *         positions of the same sequence, else 0 (the first n-1 tokens of a sequence count as novel)
 *   pi_t  positional prior max(0, 1 - p / prior_span), p = position inside the sequence
 *   score[t] = clamp(w_entropy e_t + w_novelty nu_t + w_prior pi_t, 0, 1);  a NaN e_t stays NaN.
 * One pass, one kernel: the n-gram search runs in the block that reduces the row.
 *   token_ids DEV int32 [T]; cu_seqlens DEV int32 [n_seq + 1] (cu[0] = 0, cu[n_seq] = T, unchecked on device)
 * Errors: INVALID_ARG (NULLs, negative weight, ngram outside 1..8, context or prior_span < 1), SHAPE. */
typedef struct {
  float   w_entropy, w_novelty, w_prior;
  int32_t ngram, context, prior_span;
} cwl_signal_mix;
cwl_status cwl_score_tokens_mixed(const float* logits, int64_t ld_logits, int32_t T, int32_t V,
                                  const int32_t* token_ids, const int32_t* cu_seqlens, int32_t n_seq,
                                  const cwl_signal_mix* mix, float* score, void* stream);

/* Adaptive chunker and rank-ladder selector (Sec. III-B, III-C).
 * Scores are quantised to q = floor(clamp(s,0,1) * 2^24) (NaN -> 2^24) and every mean is compared
 * as an integer sum, so the result depends on the fp32 score array only.  Per sequence a greedy
 * online walk closes the open chunk [b, e) at the first e >= b + min_len, with at least min_len
 * tokens left after it, where e - b >= max_len or the rung of [b, e) differs from the rung of the
 * look-ahead window [e, e + min_len); if fewer than 2 * min_len tokens remain, or no such e
 * exists, the chunk takes the rest of the sequence.  rung = number of thresholds the mean reaches.
 * With hi_budget = H >= 0 only the H top-rung chunks of a sequence with the largest means (earlier
 * chunk first on ties) stay on the top rung; the others step down one rung.
 *   score       DEV fp32 [T]
 *   cu_seqlens  DEV int32 [n_seq + 1], cu[0] = 0, cu[n_seq] = T, non-decreasing (unchecked on device:
 *               the caller guarantees it; empty sequences emit no chunk)
 *   table       outputs; *n_chunks <= T / min_len + n_seq entries are needed.  If capacity is
 *               too small, n_chunks is set to 0 and CWL_ERR_CAPACITY is flagged in *status_word.
 *   workspace   DEV, at least cwl_partition_workspace_bytes(T, n_seq) bytes, 16-byte aligned
 * Errors: INVALID_ARG (NULLs, bad policy, T < 0, n_seq < 0), WORKSPACE. */
size_t     cwl_partition_workspace_bytes(int32_t T, int32_t n_seq);
cwl_status cwl_partition(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                         const cwl_policy* policy, cwl_chunk_table table,
                         void* workspace, size_t workspace_bytes,
                         int32_t* status_word, void* stream);

/* Batch alignment (Sec. III-G: sequences of a batch are bucketed by complexity percentile so that chunk joins line
 * up across the batch, while each sequence still makes its own rank choices; Sec. IV-F names a batch alignment
 * controller).  The paper gives no rule; the one used here, an alternative to cwl_partition for a packed batch:
 *   1. a sequence's complexity is the mean of its quantised scores (exact integer compares); sequences are ordered
 *      by it, ascending, lower index first on ties, empty sequences first: order_pos[n] is n's position;
 *   2. bucket[n] = floor(order_pos[n] * n_buckets / n_seq): percentile bands of near-equal population;
 *   3. per bucket the scores are pooled position by position, counted from each member's start (sum of the
 *      members' quantised scores at position j, and how many members reach j);
 *   4. cwl_partition's greedy walk runs once per bucket on the pooled track, over the positions of its longest
 *      member; the mean of a span is the mean over all member tokens at those positions.  Its cuts are the
 *      bucket's shared joins;
 *   5. a member takes every shared join that leaves it at least min_len tokens; its last chunk absorbs the rest
 *      (so a chunk is shorter than max_len + min_len, as with cwl_partition);
 *   6. rung, hi_budget, rank and scale of a chunk come from the sequence's own scores, as in cwl_partition.
 * With n_buckets >= n_seq every sequence is alone in its bucket and the table equals cwl_partition's.
 *   score, cu_seqlens, policy, table, status_word   as for cwl_partition (same capacity rule and CAPACITY flag)
 *   bucket, order_pos   DEV int32 [n_seq], outputs
 *   workspace           DEV, cwl_batch_align_workspace_bytes(T, n_seq, n_buckets) bytes, 16-byte aligned
 * Errors: INVALID_ARG (NULLs, bad policy, n_buckets < 1), UNSUPPORTED (T > 2^19 tokens or n_buckets > 1024),
 * WORKSPACE, CUDA.  Scheduler-level work: nine small launches, no host synchronisation. */
size_t     cwl_batch_align_workspace_bytes(int32_t T, int32_t n_seq, int32_t n_buckets);
cwl_status cwl_batch_align(const float* score, const int32_t* cu_seqlens, int32_t n_seq, int32_t T,
                           const cwl_policy* policy, int32_t n_buckets, cwl_chunk_table table,
                           int32_t* bucket, int32_t* order_pos,
                           void* workspace, size_t workspace_bytes,
                           int32_t* status_word, void* stream);

/* Adapted projection (Sec. III-F) with the boundary-safe cross-fade (Sec. III-D):
 *   y_t = x_t W + (1 - lam_t) s_p (x_t A[:, :r_p]) B[:r_p, :] + lam_t s_c (x_t A[:, :r_c]) B[:r_c, :]
 * for row t in chunk c with predecessor p = c - 1.  Rows j = 0..window-1 of a chunk that is not
 * first of its sequence have lam = (j + 1) / (window + 1); every other row has lam = 1.
 * bf16 operands, fp32 accumulation on the tensor cores, bf16 (round-to-nearest-even) output.
 *   X DEV bf16 [T, d_in]; W DEV bf16 [d_in, d_out]; A DEV bf16 [d_in, R]; B DEV bf16 [R, d_out];
 *   Y DEV bf16 [T, d_out].  A == NULL or B == NULL or R == 0 computes the plain projection X W
 *   (table is then ignored).
 *   table       input; rows outside every chunk get no adapter.  rank[c] must lie in [0, R].
 *   workspace   DEV, at least cwl_apply_workspace_bytes(T, d_in, d_out, R) bytes, 256-byte aligned
 * Supported shapes: d_in, d_out, R multiples of 16; R <= CWL_MAX_RANK; all base pointers 16-byte
 * aligned and leading dimensions multiples of 8 elements.  Anything else is CWL_ERR_UNSUPPORTED /
 * CWL_ERR_SHAPE -- there is no slow path.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, WORKSPACE, CUDA.  T == 0 is a no-op. */
size_t     cwl_apply_workspace_bytes(int32_t T, int32_t d_in, int32_t d_out, int32_t R);
cwl_status cwl_apply(const void* X, int64_t ldx, const void* W, int64_t ldw,
                     const void* A, int64_t lda, const void* B, int64_t ldb,
                     int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                     cwl_chunk_table table, int32_t window,
                     void* Y, int64_t ldy,
                     void* workspace, size_t workspace_bytes,
                     int32_t* status_word, void* stream);

/* cwl_apply with a choice of where the cross-fade window lies (Sec. III-D asks for a short window at the join and
 * does not place it):
 *   CWL_WINDOW_CAUSAL   the first `window` rows of the incoming chunk (cwl_apply; the only placement a decode step
 *                       can use, since the incoming configuration is unknown before its chunk opens)
 *   CWL_WINDOW_CENTRED  the last floor(window/2) rows of the outgoing chunk and the first ceil(window/2) rows of the
 *                       incoming chunk (prefill: the whole table is known).  Window row i = 0..window-1, counted from
 *                       the window's first row, has lam = (i+1)/(window+1) for the incoming configuration and
 *                       1 - lam for the outgoing one.  No window at a join into the first chunk of a sequence.
 *                       Chunks between two joins should hold at least `window` rows (cwl_partition guarantees it:
 *                       window <= min_len); where a shorter chunk's two windows meet, the rows go to the join
 *                       that opened the chunk.
 * Everything else (arguments, workspace size, shape rules, errors) as cwl_apply; an unknown mode is INVALID_ARG. */
typedef enum { CWL_WINDOW_CAUSAL = 0, CWL_WINDOW_CENTRED = 1 } cwl_window_mode;
cwl_status cwl_apply_mode(const void* X, int64_t ldx, const void* W, int64_t ldw,
                          const void* A, int64_t lda, const void* B, int64_t ldb,
                          int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                          cwl_chunk_table table, int32_t window, int32_t window_mode,
                          void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes,
                          int32_t* status_word, void* stream);

/* Several adapted projections of the SAME rows in one launch (Sec. III-F: the adapter sits on every attention and
 * MLP projection; q, k, v read one activation, gate and up another).  Projection j computes
 *   Y_j = X W_j + gated (X A_j) B_j
 * exactly as cwl_apply does, with the chunk table, window, d_in and R shared by the group.  The output tiles and the
 * shrink work of all projections are scheduled together, which fills the last wave of tiles better than separate
 * calls.  Meant for prefill-sized T; decode-sized T is better served by separate cwl_apply
 * calls, whose K loop is split.
 *   proj        HOST array of n_proj descriptors (1 <= n_proj <= CWL_MAX_GROUP), copied at call time; all pointers
 *               inside are DEV.  Either every projection has A and B, or none has.
 *   workspace   DEV, at least cwl_apply_grouped_workspace_bytes(T, d_in, n_proj, d_out[], R) bytes, 256-byte aligned
 * Shape rules and errors as for cwl_apply. */
#define CWL_MAX_GROUP 4
typedef struct {
  const void* W; int64_t ldw;   /* DEV bf16 [d_in, d_out] */
  const void* A; int64_t lda;   /* DEV bf16 [d_in, R] or NULL */
  const void* B; int64_t ldb;   /* DEV bf16 [R, d_out] or NULL */
  void*       Y; int64_t ldy;   /* DEV bf16 [T, d_out] */
  int32_t d_out;
} cwl_projection;
size_t     cwl_apply_grouped_workspace_bytes(int32_t T, int32_t d_in, int32_t n_proj, const int32_t* d_out, int32_t R);
cwl_status cwl_apply_grouped(const void* X, int64_t ldx, const cwl_projection* proj, int32_t n_proj,
                             int32_t T, int32_t d_in, int32_t R, cwl_chunk_table table, int32_t window,
                             void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/* Several INDEPENDENT adapted projections in one launch (Sec. III-F: the adapter sits on every attention and MLP
 * projection; the projections of a decode step whose inputs are ready do not depend on one another).  Unlike
 * cwl_apply_grouped the projections need not read the same rows: every item has its own X, d_in, W, A, B, Y, d_out;
 * T, R, the chunk table (or the row gates) and the window are shared.  The CTA pairs are shared out among the items in
 * proportion to the bytes of their weights and every item is planned and run exactly as a cwl_apply call on that many
 * pairs would be; sharing one launch, the set-up and the drain of one item overlap the main loops of the others, and
 * consecutive batch launches chain like any other launch.  Meant for decode-sized T, where set-up and drain are a
 * large share of a launch.
 *   items       HOST array of n descriptors (1 <= n <= CWL_MAX_BATCH), copied at call time; pointers inside are DEV.
 *               An item with A == NULL or B == NULL computes X W only.
 *   gates       DEV cwl_row_gate [T] (declared below) or NULL; when set, the rows' descriptors replace the chunk table
 *   workspace   DEV, cwl_apply_batch_workspace_bytes(T, n, d_in[], d_out[], R) bytes, 256-byte aligned
 * Results equal those of n cwl_apply / cwl_apply_rows calls up to the order of fp32 sums.  Shape rules and errors as
 * for cwl_apply; UNSUPPORTED when fewer CTA pairs than items are available (cwl_set_pair_budget). */
#define CWL_MAX_BATCH 4
typedef struct {
  const void* X; int64_t ldx; int32_t d_in;     /* DEV bf16 [T, d_in] */
  const void* W; int64_t ldw;                   /* DEV bf16 [d_in, d_out] */
  const void* A; int64_t lda;                   /* DEV bf16 [d_in, R] or NULL */
  const void* B; int64_t ldb;                   /* DEV bf16 [R, d_out] or NULL */
  void*       Y; int64_t ldy; int32_t d_out;    /* DEV bf16 [T, d_out] */
} cwl_batch_item;
size_t     cwl_apply_batch_workspace_bytes(int32_t T, int32_t n, const int32_t* d_in, const int32_t* d_out, int32_t R);

/* Decode-time scheduler (Sec. III-A, III-B, III-F: scores arrive as tokens stream in, tokens are grouped as they
 * arrive, and the scheduler keeps its state from step to step): every step brings one new token per sequence.  The paper names the constraints only; the rule here is
 * causal.  Per sequence the state holds the open chunk's length and the rung it was opened on, the rung of the chunk
 * before it, and the quantised scores of the last min_len tokens.  A new token first enters that trailing window;
 * the first token of a sequence opens the first chunk on the window's rung; later, a chunk of at least min_len
 * tokens closes when it holds max_len tokens or when the window's rung differs from the rung it was opened on, and
 * the token opens a new chunk on the window's rung (one rung lower when that is the top rung and hi_budget such
 * chunks were opened already).  Rows j < window of a chunk that is not its sequence's first are cross-faded with
 * lambda = (j+1)/(window+1) (Sec. III-D).  All compares are integer (Q24 sums), so results are bit-exact.
 *   cwl_stream_state_bytes   size of the DEV state for n_seq sequences (min_len <= CWL_STREAM_MAX_MIN_LEN)
 *   cwl_stream_reset         all sequences back to "nothing seen"
 *   cwl_stream_step          score DEV fp32 [n_seq] (the new tokens' complexity scores); active DEV int32 [n_seq] or
 *                            NULL (0 = this sequence has no token this step: state untouched, its gate has rank 0);
 *                            gates DEV [n_seq], the row descriptors cwl_apply_rows consumes.  state must be 16-byte aligned.
 * Errors: INVALID_ARG (NULLs, bad policy, min_len above the limit), WORKSPACE (state missing, small or misaligned). */
#define CWL_STREAM_MAX_MIN_LEN 64
typedef struct {
  int32_t rank_in, rank_out;     /* prefix rank of the row's chunk, and of the chunk before it (used when lambda < 1) */
  float   scale_in, scale_out;   /* their gating scales */
  float   lambda;                /* weight of the row's own chunk; 1 outside a cross-fade window */
  int32_t pos_in_chunk;          /* j; -1 for an inactive sequence */
  int32_t opened;                /* 1 if this token opened a chunk */
} cwl_row_gate;
size_t     cwl_stream_state_bytes(int32_t n_seq, int32_t min_len);
cwl_status cwl_stream_reset(void* state, size_t state_bytes, int32_t n_seq, int32_t min_len, void* stream);
cwl_status cwl_stream_step(const float* score, const int32_t* active, int32_t n_seq, const cwl_policy* policy,
                           void* state, size_t state_bytes, cwl_row_gate* gates, void* stream);

/* cwl_apply with one descriptor per row instead of a chunk table (decode: every row is another sequence's newest
 * token, so rows inside a cross-fade window are blended too):
 *   y_t = x_t W + (1 - lambda_t) scale_out_t (x_t A[:, :rank_out_t]) B[:rank_out_t, :]
 *               + lambda_t scale_in_t (x_t A[:, :rank_in_t]) B[:rank_in_t, :]
 * gates DEV [T]; ranks are clamped to [0, R].  Everything else as cwl_apply (same workspace size). */
cwl_status cwl_apply_rows(const void* X, int64_t ldx, const void* W, int64_t ldw,
                          const void* A, int64_t lda, const void* B, int64_t ldb,
                          int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                          const cwl_row_gate* gates, void* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/* cwl_apply_batch: see cwl_batch_item above (declared here because it takes row gates). */
cwl_status cwl_apply_batch(const cwl_batch_item* items, int32_t n, int32_t T, int32_t R,
                           cwl_chunk_table table, const cwl_row_gate* gates, int32_t window,
                           void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream);

/* Offline construction of the rank ladder (Sec. III-C: the ladder comes from a one-off singular value decomposition
 * of the trained adapter): re-factorises a
 * trained adapter so that every prefix of the stored factors is the best adapter of its rank,
 *   A B = U diag(sigma) V^T,  A_out = U diag(sigma) [d_in, R],  B_out = V^T [R, d_out],  sigma descending,
 * by two one-sided Jacobi passes in fp64 (no d_in x d_out product, no Gram matrix).  Not on the timed path: the call
 * synchronises `stream` (once per Jacobi sweep).
 *   A DEV bf16 [d_in, R], B DEV bf16 [R, d_out]                      inputs, row-major
 *   A_out / B_out DEV bf16 or NULL; A_out_f32 [d_in, R] / B_out_f32 [R, d_out] / sigma [R] DEV fp32 or NULL (dense)
 *   workspace DEV, cwl_ladder_workspace_bytes(d_in, d_out, R) bytes, 256-byte aligned;  *sweeps HOST or NULL
 * Singular vectors are unique up to sign (and up to rotation inside equal singular values); sigma and every prefix
 * product A_out[:, :r] B_out[:r, :] are unique.
 * Errors: INVALID_ARG, UNSUPPORTED (R odd, < 2, > CWL_MAX_RANK, > d_in or > d_out), SHAPE, WORKSPACE, CUDA. */
size_t     cwl_ladder_workspace_bytes(int32_t d_in, int32_t d_out, int32_t R);
cwl_status cwl_ladder_build(const void* A, int64_t lda, const void* B, int64_t ldb,
                            int32_t d_in, int32_t d_out, int32_t R,
                            void* A_out, int64_t lda_out, void* B_out, int64_t ldb_out,
                            float* A_out_f32, float* B_out_f32, float* sigma,
                            void* workspace, size_t workspace_bytes, int32_t* sweeps, void* stream);

/* How much of the GPU the apply calls of THIS host thread plan for: at most `pairs` CTA pairs (2 SMs each; a B200
 * holds 74), 0 = all of them (the default).  Independent projections -- no one reads what another writes -- can then
 * run side by side on different streams, each on its share of the SMs, so that one call's set-up and drain (partial
 * sums handed over, outputs stored) overlap the other's weight stream; it matters for decode-sized calls, whose
 * set-up and drain are a large share of the launch (Sec. III-F puts the adapter on every attention and MLP
 * projection, and the projections of one step that read ready inputs are independent).  The budget also enters
 * cwl_apply_workspace_bytes and cwl_apply_plan-style decisions made by later calls of the thread; calls that run
 * side by side need distinct workspaces.  Budgets of concurrent calls should add up to the resident pairs or less:
 * a call's waits only make progress once all its pairs are resident (they are bounded, see CWL_ERR_TIMEOUT).
 * Errors: INVALID_ARG (pairs < 0). */
cwl_status cwl_set_pair_budget(int32_t pairs);

/* One-shot hint for the NEXT cwl_apply / cwl_apply_rows / cwl_apply_grouped call made by this host thread: the
 * region [ptr, ptr + bytes) is what the call AFTER that one will stream -- typically the weight matrix of the
 * projection that follows (weights and adapter factors are frozen at inference: Sec. III-C).  Once a CTA of the
 * hinted launch has issued its last operand load, it asks L2 for its slice of the region, so that HBM keeps
 * working while the launch combines its partial sums and stores its outputs, and while the following launch
 * sets up; that launch then finds (part of) its weights in L2.  It matters for decode-sized calls, which are
 * bound by HBM and whose drain is a large share of the launch; at most ~100 MB (less than L2) is useful.
 *   ptr   DEV, any alignment (whole 128-byte lines inside the region are requested); must stay valid until the
 *         hinted launch has completed.  The data is only read.  NULL or bytes == 0 withdraws a pending hint.
 * The hint is consumed by the next call whether or not that call launches anything; it has no effect on results.
 * Thread-local; no device work is done by this call itself. */
cwl_status cwl_prefetch_next(const void* ptr, size_t bytes);

/* The schedule cwl_apply uses for a shape when `pairs` CTA pairs can be resident (a B200 holds 74): how
 * the output is cut into column tiles (Sec. III-F leaves the kernel schedule open; this is the library's own
 * design), whether the K loop of decode-sized problems is split, and who computes the shrink X A.
 * Host-only and pure: no device is touched.  For inspection and tests.
 *   row_tiles               256-row tiles
 *   wide_width/..per_row    each row tile has wide_tiles_per_row column tiles of wide_width columns, then
 *   narrow_width/..per_row  narrow_tiles_per_row tiles of narrow_width (0, 0 if none); the last tile of a row may be ragged
 *   split_k                 pairs sharing one tile's K loop (1 = none); k_blocks_per_split 64-deep blocks each
 *   shrink_splits           splits of d_in in the shrink; shrink_items = row_tiles * shrink_splits are handed
 *                           out over the pairs (shrink_items_assigned = their total, ..max_per_pair the most one pair gets)
 *   stages                  depth of the TMA ring;  model_cost: the planner's figure for the busiest pair
 * Errors: INVALID_ARG, UNSUPPORTED (same shape rules as cwl_apply). */
typedef struct {
  int32_t pairs, row_tiles;
  int32_t wide_width, wide_tiles_per_row, narrow_width, narrow_tiles_per_row;
  int32_t split_k, k_blocks_per_split;
  int32_t shrink_splits, shrink_items, shrink_items_assigned, shrink_items_max_per_pair;
  int32_t stages;
  int64_t model_cost;
} cwl_apply_plan_info;
cwl_status cwl_apply_plan(int32_t T, int32_t d_in, int32_t d_out, int32_t R, int32_t pairs,
                          cwl_apply_plan_info* out);

/* No counterpart in the paper: a variant of cwl_apply for callers that cannot allocate device
 * memory -- code running inside another framework's memory pool, inside a region where cudaMalloc
 * is forbidden, or on a budget that was fixed before this library was loaded.  It takes no
 * workspace: the shrink partials and the gated H' live in an array of CWL_NOALLOC_SCRATCH_BYTES
 * bytes that is part of the library image (each GPU that loads the library holds it until the
 * process exits).  Inputs and outputs are still the caller's.  Same arithmetic, arguments, shape
 * rules and errors as cwl_apply (every tile keeps its whole K loop, so decode-sized problems run
 * without the split that cwl_apply would use; sums may differ in the last bit), plus:
 *   - CWL_ERR_WORKSPACE when cwl_apply_noalloc_scratch_need(T, d_in, d_out, R) exceeds
 *     CWL_NOALLOC_SCRATCH_BYTES (with R = 64 every T up to 32768 rows fits); nothing runs.
 *   - The first call on each device looks the array's device address up (once, with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array and it keeps whatever the previous call left in it.  The few
 *     words that must start at zero (per-row-tile counters and flags) are cleared by every call on its
 *     stream before the kernel; everything else that is read was written earlier in the same call.
 *     Two calls whose kernels overlap on the GPU -- different streams, or the same stream on two host
 *     threads -- race on it.  Serialise them.
 * The call allocates nothing on the device and calls no allocating CUDA or framework routine. */
#define CWL_NOALLOC_SCRATCH_BYTES (8u << 20)
size_t     cwl_apply_noalloc_scratch_need(int32_t T, int32_t d_in, int32_t d_out, int32_t R);
cwl_status cwl_apply_noalloc(const void* X, int64_t ldx, const void* W, int64_t ldw,
                             const void* A, int64_t lda, const void* B, int64_t ldb,
                             int32_t T, int32_t d_in, int32_t d_out, int32_t R,
                             cwl_chunk_table table, int32_t window,
                             void* Y, int64_t ldy, int32_t* status_word, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CWL_H */
