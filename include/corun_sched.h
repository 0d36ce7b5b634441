/*
 * Host scheduler around a CoRun engine: isolated prefill in front of the
 * fixed-shape decode iteration.
 *
 * This is the paper's scheduling wrapper (Design, "Isolated Prefill";
 * Algorithm 1 "Finding the request for isolated prefill" and Algorithm 2
 * "Scheduling isolated prefill") with the scheduler it wraps reduced to what
 * this engine needs: one decode iteration over every running request.  Two
 * queues are kept, `waiting` (requests that have not started prefill, FIFO)
 * and `running` (requests that own a slot).  One call of corun_sched_step
 * takes one scheduling decision:
 *
 *   1. the head of `waiting` starts its prefill, alone (a batch of one), iff
 *      fewer than B requests are running and the KV pool can hold its whole
 *      configured sequence (prompt + max_new_tokens) -- Algorithm 1's two
 *      admission tests; a head that does not fit blocks the queue (no request
 *      overtakes another);
 *   2. otherwise, if anything is running, one padded decode iteration for all
 *      running requests;
 *   3. otherwise nothing (idle).
 *
 * A prompt longer than one prefill chunk is prefilled chunk after chunk
 * inside that one decision (Algorithm 1 resumes a partial prefill before
 * anything else, so no decode iteration can come between the chunks anyway).
 * A request is never preempted: its pages are reserved at admission and given
 * back when it has produced max_new_tokens tokens (the first of which comes
 * from the prefill).
 *
 * The engine is reached through four callbacks, so the policy can be driven
 * against a stand-in; corun_sched_create_for_engine fills them in for a real
 * engine.  All pointers are HOST pointers.  Calls are synchronous and not
 * thread-safe.  Status codes are those of corun.h.
 */
#ifndef CORUN_SCHED_H
#define CORUN_SCHED_H

#include <stdint.h>

#include "corun.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct corun_sched corun_sched;

/* What the scheduler needs from an engine; ctx is passed back unchanged.  Each returns a corun.h
 * status (free_blocks: the number of free KV pages, or a negative status). */
typedef struct {
  int (*prefill)(void *ctx, int32_t slot, const int32_t *tokens, int32_t n, int32_t reserve_len,
                 const corun_sampling *sampling, uint64_t seed, int32_t *out_first_token);
  int (*decode_step)(void *ctx, const uint8_t *active, const uint64_t *seeds, int32_t *out_tokens);
  int (*release)(void *ctx, int32_t slot);
  int64_t (*free_blocks)(void *ctx);
} corun_sched_ops;

/* Optional: several prompts in shared prefill chunks (the signature of corun_prefill_batch). */
typedef int (*corun_sched_prefill_batch_fn)(void *ctx, int32_t n_req, const int32_t *slots, const int32_t *tokens,
                                            const int32_t *n_tokens, const int32_t *reserve_lens,
                                            const corun_sampling *samplings, const uint64_t *seeds,
                                            int32_t *out_first_tokens);

/* What one corun_sched_step did. */
enum { CORUN_SCHED_IDLE = 0, CORUN_SCHED_PREFILL = 1, CORUN_SCHED_DECODE = 2 };

/* B: slots of the engine (= the most requests that run at once); kv_block: tokens per KV page;
 * max_context: the engine's largest prompt + generated length.  The ops table is copied. */
int corun_sched_create(const corun_sched_ops *ops, void *ctx, int32_t B, int32_t kv_block, int32_t max_context,
                       corun_sched **out);
/* The same for a real engine (B, page size and max_context are the engine's). */
int corun_sched_create_for_engine(corun_engine *e, corun_sched **out);
void corun_sched_destroy(corun_sched *s);

/*
 * Batched prefill, off by default (paper, Future Work, "Batch-Invariant Kernels for Prefill": prefill
 * requests batched with each other, never with decode; an extension of Algorithms 1 and 2, not part of
 * them).  When on, a prefill decision takes the head of `waiting` exactly as before and then, in queue
 * order, every following request that (a) still finds a free slot, (b) fits the pool together with the
 * ones taken before it, and (c) fits into the padding of the chunks the requests taken so far occupy
 * anyway: a request's rows start on a multiple of tile_rows, and the number of chunks of chunk_rows rows
 * must not grow.  It stops at the first request that fails one of the three (no request overtakes
 * another), so the head is never delayed by more than the others' LM heads, and short prompts ride in
 * chunks that would have been padding.  The tokens of every request are those of isolated prefill.
 * fn NULL: the engine's corun_prefill_batch and geometry (scheduler made by _create_for_engine; chunk_rows
 * and tile_rows are then ignored); else chunk_rows >= tile_rows >= 1, chunk_rows % tile_rows == 0.
 * corun_sched_step reports the number of requests prefilled in *n_active and the first one's id.
 */
int corun_sched_enable_batched_prefill(corun_sched *s, corun_sched_prefill_batch_fn fn, int32_t chunk_rows,
                                       int32_t tile_rows);

/* Appends a request to `waiting`; the prompt is copied.  n >= 1, max_new_tokens >= 1 and
 * n + max_new_tokens <= max_context, else EINVAL.  *request_id counts up from 0 in submission order. */
int corun_sched_submit(corun_sched *s, const int32_t *prompt, int32_t n, int32_t max_new_tokens,
                       const corun_sampling *sampling, uint64_t seed, int64_t *request_id);

/* One scheduling decision (see above).  *action: CORUN_SCHED_*; *request_id: the prefilled request
 * (PREFILL; the first one of a batched prefill) else -1; *n_active: requests that took part (those
 * prefilled, the running count for a decode iteration, 0 when idle).  An engine error is returned as is and
 * leaves the queues as they were before the call.  One case ends a request without serving it: when nothing
 * runs (so the whole pool is free) and the head of `waiting` still does not fit, it can never fit; the step
 * then removes it, marks it finished with no tokens, sets *request_id to it and returns CORUN_ENOSPACE (action
 * IDLE), so that the requests behind it are not blocked for good. */
int corun_sched_step(corun_sched *s, int32_t *action, int64_t *request_id, int32_t *n_active);

/* Tokens produced so far by a request (at most cap are copied; *n_tokens is the full count) and
 * whether it has finished.  Requests stay queryable until the scheduler is destroyed. */
int corun_sched_poll(corun_sched *s, int64_t request_id, int32_t *tokens, int32_t cap, int32_t *n_tokens,
                     int32_t *finished);
/* The slot a running request occupies (-1 when it is waiting or finished). */
int corun_sched_slot_of(corun_sched *s, int64_t request_id, int32_t *slot);
int corun_sched_counts(corun_sched *s, int32_t *n_waiting, int32_t *n_running);

#ifdef __cplusplus
}
#endif
#endif
