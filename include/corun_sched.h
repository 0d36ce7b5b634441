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

/* What one corun_sched_step did. */
enum { CORUN_SCHED_IDLE = 0, CORUN_SCHED_PREFILL = 1, CORUN_SCHED_DECODE = 2 };

/* B: slots of the engine (= the most requests that run at once); kv_block: tokens per KV page;
 * max_context: the engine's largest prompt + generated length.  The ops table is copied. */
int corun_sched_create(const corun_sched_ops *ops, void *ctx, int32_t B, int32_t kv_block, int32_t max_context,
                       corun_sched **out);
/* The same for a real engine (B, page size and max_context are the engine's). */
int corun_sched_create_for_engine(corun_engine *e, corun_sched **out);
void corun_sched_destroy(corun_sched *s);

/* Appends a request to `waiting`; the prompt is copied.  n >= 1, max_new_tokens >= 1 and
 * n + max_new_tokens <= max_context, else EINVAL.  *request_id counts up from 0 in submission order. */
int corun_sched_submit(corun_sched *s, const int32_t *prompt, int32_t n, int32_t max_new_tokens,
                       const corun_sampling *sampling, uint64_t seed, int64_t *request_id);

/* One scheduling decision (see above).  *action: CORUN_SCHED_*; *request_id: the prefilled request
 * (PREFILL) else -1; *n_active: requests that took part (1 for a prefill, the running count for a
 * decode iteration, 0 when idle).  An engine error is returned as is and leaves the queues as they
 * were before the call. */
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
