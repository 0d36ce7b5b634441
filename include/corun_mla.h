/*
 * Multi-head latent attention (MLA) for one query token per row at decode time, in the absorbed form, for
 * NVIDIA B200 (sm_100a).  The contraction runs on the warp-level tensor path (mma.sync m16n8k16, fp16 operands,
 * fp32 accumulation): one CTA per row and chunk of 512 cached tokens streams the chunk in tiles of 64 tokens
 * through shared memory with an online softmax; the chunks of a row are combined in ascending order.  (A plain
 * fp32 FMA kernel over splits of 128 tokens serves the shapes the tensor path does not take.)
 *
 * The paper evaluates an MLA model (Evaluation, "Setup") and turns decode-time Split-KV off because its split
 * count depends on the batch (Design, "Fixed-Shape Batched Decode"); here, as in the dense attention kernel,
 * the split size is fixed and the split count depends on the row's own context length only, so a row's
 * result does not depend on the other rows of the step.
 *
 * Per cached token the cache holds the latent c_t [d_c] followed by the shared rotary key r_t [d_r] (fp16,
 * d_c + d_r values per token); all n_heads query heads of a row share it.  With the up-projections absorbed
 * into the query (q_lat[h] = W_uk[h]^T q_nope[h]) a head's scores and output are
 *     s_{h,t} = (q_lat[h] . c_t + q_rope[h] . r_t) * scale,   p_h = softmax_t(s_h),   o_lat[h] = sum_t p_{h,t} c_t
 * (the caller applies W_uv[h] to o_lat[h]).  All pointers are DEVICE pointers; the call is asynchronous on the
 * given stream.  Status codes are those of corun.h.
 */
#ifndef CORUN_MLA_H
#define CORUN_MLA_H

#include <stdint.h>

#include "corun.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Floats of workspace corun_mla_attend needs for B rows of at most max_context cached tokens. */
int64_t corun_mla_workspace_floats(int32_t B, int32_t n_heads, int32_t d_latent, int32_t max_context);

/*
 *   q_lat   fp32 [B, n_heads, d_latent]      q_rope  fp32 [B, n_heads, d_rope]
 *   cache   fp16 [B, max_context, d_latent + d_rope] (row b uses its first ctx[b] tokens)
 *   ctx     int32 [B]: cached tokens per row, 0 = padding row (its output is left alone); a value above
 *           max_context is treated as max_context (nothing past a row's cache is read)
 *   o_lat   fp32 [B, n_heads, d_latent]
 *   ws      corun_mla_workspace_floats(...) floats
 * n_heads 1..16 (a multiple of 4), d_latent a multiple of 64 up to 512, d_rope a multiple of 8 up to 64
 * (cache rows are then 16-byte aligned).
 * operand_pairs  1: the fp32 queries and softmax weights enter the tensor cores as fp16 hi + lo pairs (two
 *                   instructions per tile; results agree with fp64 to ~1e-5);
 *                0: as single fp16 values, the precision of a conventional fp16 attention kernel, at half the
 *                   tensor work (needs d_rope a multiple of 16; the weight sum runs over the rounded weights).
 *                Either way a row's result depends on the row alone.
 * Errors: EINVAL, ECUDA.
 */
int corun_mla_attend(const float *q_lat, const float *q_rope, const void *cache, const int32_t *ctx, int32_t B,
                     int32_t n_heads, int32_t d_latent, int32_t d_rope, int32_t max_context, float scale, float *o_lat,
                     float *ws, int32_t operand_pairs, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
