/*
 * Mixture-of-Experts feed-forward block at decode time, position-invariant by
 * construction, for NVIDIA B200 (sm_100a).
 *
 * The paper evaluates Mixture-of-Experts models (Evaluation, "Setup") and
 * observes, in its comparison with LLM-42, that a small router perturbation
 * changes the selected experts.  In the fixed-shape decode iteration (Design,
 * "Fixed-Shape Batched Decode") the number of rows that pick an expert depends
 * on the co-tenants, so a per-expert GEMM whose TILE SHAPE followed that number
 * would compute a row differently from step to step.  Here every shape is a
 * function of the padded row count B alone.  For B padded rows x [B, H]:
 *
 *   router   logits = x Wr^T, p = softmax over all E experts, S = top_k by p
 *            (ties to the lower expert id), weights p_e as they are or, on
 *            request, renormalised over the selected ones; shared experts always
 *            on with weight 1;
 *
 * up to 64 padded rows, without groups (every row through every expert):
 *   GEMM 1   [B, H] x all experts' gate and up rows: [B, (E + S) * 2F];
 *   SwiGLU   h[r, e*F + f] = w[r, e] * silu(gate) * up, exactly 0 for the
 *            experts row r did not select;
 *   GEMM 2   y = h Wd_cat^T with K = (E + S) * F: the sum over a row's experts
 *            happens inside the accumulator, in ascending expert id (shared
 *            experts last), unselected experts contributing exact zeros.
 *   All experts' weights are streamed once per call whatever was selected: the
 *   padding the paper's title refers to, applied to experts.
 *
 * above 64 padded rows (where two MMAs per k-slice for the hi and lo halves of
 * 128 rows would keep the tensor pipe as busy as the weight stream), grouped:
 *   grouping the rows that selected expert e, in ascending row order, fill blocks
 *            of exactly 64 rows (the last one padded); experts ascending;
 *   gather   the rows' hi / lo activations into their blocks;
 *   GEMM 1   per block: [64, H] x the expert's gate and up rows, w[r, e] *
 *            silu(gate) * up in the epilogue;
 *   GEMM 2   per block: [64, F] x the expert's down projection, fp32;
 *   combine  y[r] = the row's experts' results added in ascending expert id
 *            (shared experts last).
 *   The block shape, the tiles and the K order are the same for every block and
 *   every step; an accumulator row is computed from its own activation row only,
 *   so neither the row's place in its block nor what else the block holds
 *   reaches its result.  Experts nobody selected are not streamed.
 *
 * Either way the GEMMs are the library's decode GEMM (fixed tiles and K order
 * for a given B), so a row's result depends on its own x only: not on its row
 * index, not on what the other rows are or select.
 *
 * All data pointers are DEVICE pointers; calls are asynchronous on the stream
 * given at creation except where stated.  Status codes are those of corun.h.
 */
#ifndef CORUN_MOE_H
#define CORUN_MOE_H

#include <stdint.h>

#include "corun.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct corun_moe corun_moe;

typedef struct {
  int32_t hidden;      /* H, multiple of 64 */
  int32_t n_experts;   /* E routed experts, 1..256 */
  int32_t top_k;       /* 1..min(E, 16) */
  int32_t expert_ffn;  /* F, multiple of 64; 2F a multiple of 4 */
  int32_t n_shared;    /* always-on experts of the same size, >= 0 */
  int32_t renormalize; /* 0: the selected probabilities as they are; 1: divided by their sum (added in
                          descending-probability order) */
} corun_moe_shape;

/*
 * Weights, bf16, row-major, borrowed until corun_moe_destroy:
 *   router   [E, H]
 *   gate_up  [(E + n_shared) * 2F, H]: block e = expert e (shared experts behind the routed ones);
 *            its rows 0..F-1 are the gate projection, F..2F-1 the up projection
 *   down     [H, (E + n_shared) * F]: columns e*F .. e*F+F-1 are expert e's down projection
 * B: padded rows per call (1..256).  Synchronous.  Errors: EINVAL, ENOMEM, ECUDA.
 */
int corun_moe_create(const corun_moe_shape *shape, const void *router, const void *gate_up, const void *down,
                     int32_t B, void *cuda_stream, corun_moe **out);
void corun_moe_destroy(corun_moe *m);

/*
 * y = MoE(x) for all B rows.  x, y: fp32 [B, H] (y may not alias x; y must start on a 16-byte boundary, x on a
 * 4-byte one: EINVAL otherwise, before anything is launched).  experts (int32 [B, top_k], by
 * descending probability) and probs (fp32 [B, top_k]) receive the routing when not NULL.
 * Asynchronous; corun_moe_sync waits and reports a device-side timeout (ETIMEOUT).
 */
int corun_moe_forward(corun_moe *m, const float *x, float *y, int32_t *experts, float *probs);
int corun_moe_sync(corun_moe *m);
/* Bytes of expert and router weights one call streams (the roofline's numerator). */
int64_t corun_moe_weight_bytes(const corun_moe *m);
/* Kernels launched by one corun_moe_forward. */
int corun_moe_launches(const corun_moe *m);

#ifdef __cplusplus
}
#endif
#endif
