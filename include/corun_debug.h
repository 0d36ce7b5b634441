/*
 * corun_debug.h -- test and measurement accessors of libcorun.so.
 *
 * None of these is part of the serving path (paper: Design; the calls a server makes are in corun.h).  They
 * exist so that the tests can compare the engine with the oracle at sizes the oracle cannot prefill (cache
 * read / write, adopting a slot), check that eager launches equal the graph replay, run single kernels
 * against their definitions, and so that bench.py can time each kernel kind with CUDA events.  Same
 * conventions as corun.h: plain pointers and sizes, 0 or a negative corun_status, no exceptions.
 *
 * The kernel timelines (globaltimer stamps inside the GEMM and attention kernels) are compiled in only when
 * the library is built with -DCORUN_BUILD_DEBUG (python -m paper_2608_14376_b200.build with
 * CORUN_BUILD_DEBUG=1 in the environment): the serving build carries neither the stamped kernel
 * instantiations nor their readers.
 */
#ifndef CORUN_DEBUG_H_
#define CORUN_DEBUG_H_

#include "corun.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Reads / writes n cached positions [pos0, pos0+n) of one layer as fp32 rows of
 * n_kv_heads*head_dim (host).  Writing beyond the current context length
 * extends it (up to reserve_len); values are rounded to the cache's fp16. */
int corun_debug_kv_read(corun_engine *e, int32_t slot, int32_t layer, int32_t pos0, int32_t n, float *k, float *v);
int corun_debug_kv_write(corun_engine *e, int32_t slot, int32_t layer, int32_t pos0, int32_t n, const float *k,
                         const float *v);
/* Occupies an empty slot without running a prefill: reserves pages, sets the
 * context length to n_ctx (cache contents undefined until written with
 * corun_debug_kv_write), the pending token and the sampling state. */
int corun_debug_adopt(corun_engine *e, int32_t slot, int32_t n_ctx, int32_t reserve_len, int32_t pending_token,
                      const corun_sampling *sampling, int32_t step);
/* Bench set-up: fills cached positions [0, n_ctx) of every layer of an occupied slot
 * with seeded N(0, std^2) values generated on the device and sets its context length. */
int corun_debug_kv_fill(corun_engine *e, int32_t slot, int32_t n_ctx, float std, uint64_t seed);
/* Times one kernel kind of the decode program in isolation, on the engine's stream,
 * with CUDA events: `reps` launches rotating over the layers' weights (so that L2
 * cannot hold them), after a short warm-up; *avg_ms = mean duration of one launch.
 * kind: 0 QKV GEMM, 1 O GEMM, 2 gate-up GEMM, 3 down GEMM, 4 LM-head GEMM (+ partial
 * fix-up), 5 attention (split + combine), 6 residual + RMSNorm, 7 RoPE + KV append,
 * 8 SwiGLU (none where the gate / up GEMM applies it), 9 sampler; engines with multi-head latent attention:
 * 5 = the latent attention (splits + combine), 7 = latent RMSNorm + rotary key + cache append + query parts,
 * 10 = grouped key up-projection, 11 = grouped value up-projection + split; engines with expert layers:
 * 2, 3, 6, 8 on the expert layers, 12 = router; where the decode program runs the expert layers in their grouped
 * form (more than 64 padded rows): 2 = per-group gate / up GEMM (+ SwiGLU kernel where it is not in the epilogue),
 * 3 = per-group down GEMM + the sum over each row's experts, 13 = grouping + gather, all on the groups of the last
 * step's last layer.  EINVAL for a kind the engine does not have.
 * Uses the rows of the last decode step; overwrites
 * intermediate buffers (not the cache beyond each active slot's next position). */
int corun_debug_time_kernel(corun_engine *e, int32_t kind, int32_t reps, float *avg_ms);
/* Copies the first n floats of an intermediate buffer of the decode program to the host, as left by
 * the last decode step: which = 0 rotated queries [B, nq*hd]; 1 attention split partials
 * [B][nq][max_splits][hd]; 2 their (max, sum) pairs [B][nq][max_splits][2] (base-2 domain);
 * 3 the residual stream [B, hidden]; 4 / 5 the attention output's bf16 hi / lo halves [BN, nq*hd] as raw
 * memory (two bf16 per float); 6 the O-projection's direct output [B, hidden]; 7 the GEMM partial workspace. */
int corun_debug_read(corun_engine *e, int32_t which, float *out, int64_t n);
/* eager != 0: launch the decode kernels one by one instead of replaying the graph. */
int corun_debug_set_eager(corun_engine *e, int32_t eager);
/* Stand-alone run of the decode GEMM: out[r, n] = sum_k W[n, k] * X[r, k] with X
 * fp32 [R, K] (device), W bf16 [N, K] (device), out fp32 [R, N] (device); R <= 256,
 * K % 64 == 0; `out` and `W` must start on a 16-byte boundary, `X` on a 4-byte one
 * (CORUN_EINVAL otherwise, before anything is launched).  Uses the engine-independent
 * kernel path (split activations, tcgen05 MMA, fixed K order). */
int corun_debug_gemm(const void *W, int32_t N, int32_t K, const float *X, int32_t R, float *out, void *cuda_stream);
/* R(seed, t) as the engine computes it (top 24 bits of the first Philox word), on the device. */
int corun_debug_variate(uint64_t seed, uint64_t t, uint32_t *out_u24 /* host */);
/* Runs the engine's sampler on host logits rows [n_rows, vocab] (copied to the device). */
int corun_debug_sample(const float *logits, int32_t n_rows, int32_t vocab, const corun_sampling *sampling,
                       const uint32_t *u24, int32_t *out_tokens);

/* Makes a bounded device-side wait run out, harmlessly: a one-CTA kernel waits, with the wait routine every
 * kernel of the library uses and the given limit (1 us .. 100 ms), on a barrier nothing arrives at; the wait
 * gives up, the kernel records it and returns normally, and the call returns CORUN_ETIMEOUT (CORUN_OK would mean
 * the wait did not run out).  The context stays usable.  (Paper: none; failure detection of this library.) */
int corun_debug_wait_probe(uint64_t limit_ns, void *cuda_stream);
/* The index checks the kernels apply in a library built with -DCORUN_CHECKED (csrc/checks.cuh), evaluated on the
 * host: returns 1 (in range) or 0.  kind 0: (slot, n_slots, pos, max_blocks, kv_block); 1: (page, pool_blocks);
 * 2: attention item (row, n_rows, kv head, n_kv, split, context, tokens per split); 3: GEMM workspace slot
 * (cta, slot, grid).  Unused arguments are ignored.  Needs no GPU. */
int corun_debug_check_index(int32_t kind, int64_t a, int64_t b, int64_t c, int64_t d, int64_t e, int64_t f, int64_t g);

/*
 * Micro-benchmark of three reductions with a tiling fixed for every batch size against one that adapts to it
 * (paper, Introduction and the operator comparison of its motivation: batch-invariant kernels pay for one tiling
 * everywhere; this library's path only keeps the tiling fixed for its one padded shape).  Not part of the
 * decode path.
 *   kind     0 RMSNorm of every row of x [R, N] -> y [R, N]; 1 row softmax, same shapes; 2 sum over the R rows
 *            -> y [N]
 *   variant  0 fixed (one CTA per row, or per 256 columns with the rows added in ascending order: a result's
 *            bits do not depend on R); 1 adaptive (few rows: a row split over a cluster of up to 8 CTAs; kind 2:
 *            the rows split over CTAs whose partial sums meet in atomics, so the order is not fixed at all)
 *   x, y     device, fp32, 16-byte aligned; N a multiple of 32
 *   avg_us   host: mean duration of `reps` launches after one warm-up launch (CUDA events on the stream)
 *   tiling   host, may be NULL: CTAs per row (kinds 0, 1) or row chunks (kind 2) that were used
 * Synchronous.  Errors: EINVAL, ECUDA.
 */
int corun_debug_microbench(int32_t kind, int32_t variant, const float *x, int32_t R, int32_t N, float *y, int32_t reps,
                           float *avg_us, int32_t *tiling, void *cuda_stream);

#ifdef CORUN_BUILD_DEBUG
/* Runs GEMM `kind` (0 QKV, 1 O, 2 gate-up, 3 down, 4 LM head) of the decode program on one layer's
 * weights three times and returns the last launch's per-CTA timeline: stamps[cta*8 + i] (host, room for
 * 8 * 256 values) are globaltimer nanoseconds at: 0 kernel entry, 1 set-up done, 2 first TMA issued,
 * 3 last TMA issued, 4 first stage landed, 5 last MMA issued, 6 last accumulator complete, 7 epilogue done. */
int corun_debug_gemm_trace(corun_engine *e, int32_t kind, int32_t layer, uint64_t *stamps, int32_t *n_ctas);
/* With CORUN_TRACE_STEP=1 in the environment at corun_init, every layer GEMM of the decode program records
 * its per-CTA timeline (the 8 stamps of corun_debug_gemm_trace) on every step; this copies the last step's
 * stamps, [4 * n_layers][n_sms][8] values (n must equal that count), to the host. */
int corun_debug_step_trace(corun_engine *e, uint64_t *stamps, int64_t n);
/* Runs the attention of one layer twice on the rows of the last decode step and returns the second launch's
 * timeline: stamps[(cta*64 + k)*4 + i] (host, room for 256*64*4 values), globaltimer ns of the CTA's k-th item
 * (k < 64): 0 load issued, 1 item landed (seen by its consumer group), 2 the group starts on it, 3 released. */
int corun_debug_attn_trace(corun_engine *e, int32_t layer, uint64_t *stamps, int32_t *n_ctas);
#endif /* CORUN_BUILD_DEBUG */

#ifdef __cplusplus
}
#endif
#endif /* CORUN_DEBUG_H_ */
