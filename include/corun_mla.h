/*
 * Multi-head latent attention (MLA) for one query token per row at decode time, in the absorbed form, over a
 * paged latent cache, for NVIDIA B200 (sm_100a): tcgen05 MMAs with TMEM accumulators, the cache streamed by TMA
 * straight from the page pool (csrc/mla_paged.cu).
 *
 * The paper evaluates an MLA model (Evaluation, "Setup") and turns decode-time Split-KV off because its split
 * count depends on the batch (Design, "Fixed-Shape Batched Decode"); here, as in the dense attention kernel,
 * the split size is fixed (256 tokens) and the split count depends on the row's own context length only, so a
 * row's result does not depend on the other rows of the step, nor on where its pages lie in the pool.
 *
 * Per cached token the cache holds the latent c_t [d_c] followed by the shared rotary key r_t [d_r] (fp16,
 * d_c + d_r values per token); all n_heads query heads of a row share it.  With the up-projections absorbed
 * into the query (q_lat[h] = W_uk[h]^T q_nope[h]) a head's scores and output are
 *     s_{h,t} = (q_lat[h] . c_t + q_rope[h] . r_t) * scale,   p_h = softmax_t(s_h),   o_lat[h] = sum_t p_{h,t} c_t
 * (the caller applies W_uv[h] to o_lat[h]).  The fp32 queries and softmax weights enter the tensor cores as fp16
 * hi + lo pairs; results agree with fp64 to ~1e-5.  All pointers are DEVICE pointers; the call is asynchronous on
 * the given stream.  Status codes are those of corun.h.
 */
#ifndef CORUN_MLA_H
#define CORUN_MLA_H

#include <stdint.h>

#include "corun.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Floats of workspace corun_mla_attend needs for B rows of at most max_context = max_blocks * 16 cached tokens. */
int64_t corun_mla_workspace_floats(int32_t B, int32_t n_heads, int32_t d_latent, int32_t max_context);

/*
 *   q_lat        fp32 [B, n_heads, d_latent]      q_rope  fp32 [B, n_heads, d_rope]   (both 16-byte aligned)
 *   pool         fp16 [pool_pages][16 tokens][d_latent + d_rope]: the page pool (16-byte aligned).  Every value
 *                of a page that is listed for a row must be finite, also at positions beyond the row's context
 *                (they are multiplied by zero weights)
 *   block_table  int32 [B, max_blocks]: row b's page for tokens 16 i .. 16 i + 15 is block_table[b][i]
 *   ctx          int32 [B]: cached tokens per row, 0 = padding row (its output is left alone); a value above
 *                max_blocks * 16 is treated as that
 *   o_lat        fp32 [B, n_heads, d_latent] (16-byte aligned)
 *   ws           corun_mla_workspace_floats(B, n_heads, d_latent, max_blocks * 16) floats (16-byte aligned)
 * B 1..1024, n_heads 1..16, d_latent 64, 128, 256 or 512, d_rope a multiple of 8 up to 64, scale > 0.
 * Errors: EINVAL, ECUDA.  A bounded device-side wait that expires is recorded in the workspace:
 * corun_mla_sync waits for the stream and returns ETIMEOUT in that case.
 */
int corun_mla_attend(const float *q_lat, const float *q_rope, const void *pool, int64_t pool_pages, const int32_t *block_table,
                     int32_t max_blocks, const int32_t *ctx, int32_t B, int32_t n_heads, int32_t d_latent, int32_t d_rope,
                     float scale, float *o_lat, float *ws, void *cuda_stream);
int corun_mla_sync(const float *ws, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
