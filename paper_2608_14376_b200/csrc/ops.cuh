// Launchers of the non-GEMM kernels of the decode / prefill row program.
// A "row" is one query token: in decode the rows are the slots in the order prepare_rows gives them (the slots
// with a request this step first; Rows::slot names a row's slot), in prefill the rows are consecutive prompt
// positions of one slot.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm.cuh"

namespace corun {

constexpr int KV_BLOCK = 16;      // tokens per page
constexpr int ATT_SPLIT = 128;    // tokens per attention split (fixed; count = f(own context))

// Per-row metadata (device arrays of length R).
struct Rows {
  const int *token;    // token fed to the row
  const int *pos;      // position of that token = tokens cached before it
  const int *active;   // 0 = padding row
  const int *slot;     // whose block table the row uses
  int R;
};

// Offsets (in halfs) inside one page: keys as [head][token][dim], then values the same way.  The scores
// contract over dims (the key tile is a K-major operand); the weighted values contract over tokens, for which
// the value tile, read through the same kind of TMA box as the keys (rows of 128 bytes), is an MN-major operand.
__host__ __device__ inline size_t kv_k_off(int hd, int g, int tok, int dim) {
  return ((size_t)g * KV_BLOCK + tok) * hd + dim;
}
__host__ __device__ inline size_t kv_v_off(int n_kv, int hd, int g, int tok, int dim) {
  return (size_t)n_kv * KV_BLOCK * hd + ((size_t)g * KV_BLOCK + tok) * hd + dim;
}

struct KvLayout {
  __half *pool;            // [layer][page][ K: [n_kv][16][hd] | V: [n_kv][16][hd] ]
  const int *block_table;  // [n_slots][max_blocks]
  int max_blocks, n_kv, hd;
  size_t layer_stride;     // halfs per layer
  long long pool_blocks;   // pages per layer
  int n_slots;             // rows of the block table
};

struct SampleArgs {
  const float *logits;     // [R, V]
  int V;
  const int *do_sample;    // per row: 0 skip, 1 sample
  const float *temperature, *top_p;  // per row
  const uint64_t *seed;    // per row
  const int *step;         // per row: t of R(seed, t)
  const uint32_t *u24_override;  // optional per-row variate (debug); nullptr = Philox
  int *out_token;          // per row (untouched when skipped)
};

// h = E[token] (first = 1) or h += GEMM result (first = 0); then RMSNorm with
// gains g -> bf16 hi/lo pair.
cudaError_t launch_resid_norm(float *h, int H, const __nv_bfloat16 *embed, const Rows &rows, const GemmOut *prev,
                              const __nv_bfloat16 *gains, float eps, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                              cudaStream_t st);
// RoPE on q and k, q -> q_out fp32 [R, nq*hd], k/v -> pages (fp16) at the row's position.
cudaError_t launch_qkv_post(const GemmOut &qkv, const Rows &rows, const float2 *rope_tab, int nq, const KvLayout &kv,
                            int layer, float *q_out, int *d_status, cudaStream_t st);
// Split-KV paged attention partials and, in a second kernel, their fixed-order combine -> bf16 hi/lo
// [R, nq*hd] (rows that are not active keep what they held).  pool_count: one int, zero before the launch (not reset by it): the items beyond the
// CTAs' fixed stretches are drawn through it.  reuse: 1 when the rows are the consecutive tokens of one
// request in one slot (a prefill chunk): launch_attention_prefill runs instead; 2 for the ablation in which a
// CTA takes whole (row, kv head) pairs (the work list then carries the pair table); else 0.
// tmK / tmV: tensor maps over this layer's pages: keys as rows of hd halfs with a [16, 64] box (128-byte
// swizzle), and the values, cached alike, through the same view; see attention.cu.
// work / n_work: the step's (row, kv head, split) items from launch_attn_worklist (the same for every layer);
// grid_ctas: persistent CTAs to launch (one per SM).
cudaError_t launch_attention(const CUtensorMap &tmK, const CUtensorMap &tmV, const float *q, const Rows &rows, int nq,
                             const KvLayout &kv, int layer, int max_splits, const int *work, const int *n_work,
                             int grid_ctas, float *part_acc, float *part_ml, int *pool_count,
                             __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int reuse, int *d_status, cudaStream_t st,
                             unsigned long long *trace = nullptr);   // optional [grid][64][8] stamps (debug)
// n_work: 2 + 2 * rows * n_kv ints (item count, pair count, then the pairs' (first item, split count) when
// whole_pairs is set: the ablation in which a CTA takes whole (row, kv head) pairs).  Also zeroes the
// launches' pool counters.
cudaError_t launch_attn_worklist(const Rows &rows, int n_kv, int *work, int *n_work, int *pool_counts,
                                 int n_pool_counts, int whole_pairs, cudaStream_t st);
// Causal attention of a prefill chunk (rows = consecutive tokens of one request, all of one slot): query
// tiles share the key / value tiles they read; writes the bf16 hi/lo output directly (attention_prefill.cu).
cudaError_t launch_attention_prefill(const CUtensorMap &tmK, const CUtensorMap &tmV, const float *q, const Rows &rows,
                                     int nq, const KvLayout &kv, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                     int *d_status, cudaStream_t st);
cudaError_t attention_prepare();   // opts the kernels into their shared-memory size (idempotent)
// y = silu(gate) * up from the gate-up GEMM result -> bf16 hi/lo [R, F].
cudaError_t launch_swiglu(const GemmOut &gu, int R, int F, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, cudaStream_t st);
// x fp32 [R, K] -> bf16 hi/lo.
cudaError_t launch_split(const float *x, int R, int K, __nv_bfloat16 *hi, __nv_bfloat16 *lo, cudaStream_t st);
cudaError_t launch_sampler(const SampleArgs &a, int R, cudaStream_t st, bool pdl = false);
// decode bookkeeping
// The step's inputs (active mask, seeds) and results (tokens, status word) live in pinned host memory and are
// read / written by these two kernels through its device mapping: no copy nodes around the step.
cudaError_t launch_prepare_rows(const uint8_t *active_mask, const uint64_t *seeds_in, uint64_t *seeds_out, const int *in_use,
                                const int *ctx_len, const int *pending, const float *temp, const float *top_p, const int *step,
                                int B, int *row_token, int *row_pos, int *row_active, int *row_slot, int *do_sample,
                                float *row_temp, float *row_top_p, int *row_step, int *slot_row, int *row_blocks,
                                cudaStream_t st);   // rows = the slots with a request first; row_blocks: see GemmPlan::row_blocks
cudaError_t launch_advance(const int *slot_row, const int *row_active, const int *sampled, int B, int *ctx_len, int *step,
                           int *pending, int *out_tokens, const int *status_in, int *status_out, cudaStream_t st);
// debug cache access (fp32 rows of n_kv*hd)
cudaError_t launch_kv_copy(const KvLayout &kv, int layer, int slot, int pos0, int n, float *k, float *v, int write,
                           cudaStream_t st);
// fills cached positions [0, n) of every layer of a slot with seeded N(0, std^2) values (bench set-up)
cudaError_t launch_kv_fill(const KvLayout &kv, int n_layers, int slot, int n, float std, uint64_t seed, cudaStream_t st);
cudaError_t launch_variate(uint64_t seed, uint64_t t, uint32_t *out, cudaStream_t st);

}  // namespace corun
