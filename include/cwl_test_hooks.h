/*
 * cwl_test_hooks.h -- declarations that exist only in the TEST build of the library (libcwl_hooks.so, the same
 * sources compiled with -DCWL_TEST_HOOKS).  The shipped libcwl.so has none of this.
 */
#ifndef CWL_TEST_HOOKS_H
#define CWL_TEST_HOOKS_H

#include "cwl.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Test hook for the failure path of cwl_apply and its variants.  Every device-side wait (mbarrier, H' flag, split-K
 * counter) is bounded; when one runs out the CTA raises CWL_ERR_TIMEOUT in *status_word (bit 1 << CWL_ERR_TIMEOUT),
 * drains its copies, frees its tensor memory and returns, so the context stays usable.  This call sets the limit
 * (ns; <= 0 restores the default of 2 s) and, with withhold_publish != 0, makes the shrink never publish H', so that
 * the waits on it run out.  Process-wide (two atomics). */
void cwl_debug_set(int64_t wait_limit_ns, int32_t withhold_publish);

/* Read-bandwidth ceiling of one decode-sized launch: 148 CTAs (one per SM) stream [ptr, ptr + bytes) once, each its
 * slice, through a 192 KB shared-memory ring with contiguous 16 KB bulk copies, and drop the data.  No tensor-core
 * work, no outputs.  Launched like the apply kernel (its set-up may overlap the tail of the launch ahead of it).
 *   ptr  DEV, 128-byte aligned; bytes >= 148 * 16 KB (whole 16 KB pieces per CTA are read).
 * Errors: INVALID_ARG, CUDA; a wait that runs out flags CWL_ERR_TIMEOUT in *status_word. */
cwl_status cwl_probe_read(const void* ptr, size_t bytes, int32_t* status_word, void* stream);

/* The same read with the apply kernel's second source mixed in: `ctas` CTAs (1..148) each stream their slice of
 * [ptr, ptr + bytes) in 16 KB pieces and, with every piece, copy hot_piece bytes from [hot, hot + hot_bytes) at an offset
 * that is the same in every CTA (as the rows of X are for every column tile), into one ring slot; 192 KB of slots.
 *   ptr, hot  DEV, 128-byte aligned; hot_piece a multiple of 16, 16..32768; hot_bytes >= hot_piece.
 * Errors: INVALID_ARG, CUDA; a wait that runs out flags CWL_ERR_TIMEOUT in *status_word. */
cwl_status cwl_probe_read_mix(const void* ptr, size_t bytes, const void* hot, size_t hot_bytes, uint32_t hot_piece,
                              int32_t ctas, int32_t* status_word, void* stream);

/* Device timeline of one CTA pair of the apply kernels (any cwl_apply* call made afterwards).  The leader CTA of
 * pair `pair` (blockIdx.x / 2 of the launch; in a batch launch pairs are numbered through all projections) writes
 * %globaltimer readings (ns, 32 ns granularity) into slots[0..1023]; every launch overwrites the slots, so read them
 * after the launch of interest.  slots == NULL or pair < 0 switches tracing off.
 *   slots  DEV, 1024 int64, zeroed by the caller.
 *   [0] kernel entered   [1] the launch ahead in the stream has finished (griddepcontrol.wait returned)
 *   [2] last accumulator committed by the MMA issuer   [5] epilogue saw the last accumulator
 *   [3] epilogue left its item loop   [4] CTA barrier of the teardown passed
 *   split-K hand-over: [6] partial sums stored  [7] all contributors arrived  [8] their sums copied in  [9] reduced and staged
 *   shrink epilogue:   [11] partial sums stored and fenced  [12] arrival counted  [13] reduced (last arriver only)  [14] fenced
 *                      (last arriver, inside the reduce: [17] fence passed  [18] all partial sums loaded and added)
 *   [15],[16] producer: wait for the H' flag begins / ends
 *   [19],[20],[21] producer: past the wait for the launch ahead, first work item decoded, first ring slot free
 *   K block i of the pair (running count over its items, i < 290): [100+i] loads issued, [400+i] operands landed
 *   (MMA issuer's wait returned), [700+i] MMAs issued and committed.
 * Errors: CUDA. */
cwl_status cwl_trace_set(long long* slots, int32_t pair);

#ifdef __cplusplus
}
#endif
#endif /* CWL_TEST_HOOKS_H */
