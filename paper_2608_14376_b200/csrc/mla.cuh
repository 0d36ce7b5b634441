// Launchers of the multi-head latent attention (MLA) kernels for the engine's row program (mla_layer.cu,
// mla_paged.cu).  A row is one query token; its cached tokens are the latent vectors c_t and rotary keys r_t of
// its slot, [rank + rope] fp16 per token in pages of 16 tokens.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "gemm.cuh"
#include "ops.cuh"

namespace corun {

struct MlaDims {
  int nh, rank, nope, rope, vh;   // heads, latent width, per-head no-rope / rope query widths, value width
};

// One layer's latent pages and how a row finds its own.
// run = 1: the pool is [page][16 tokens][rank + rope] (a token's values contiguous).
// run = 4: pages come in aligned runs of four (blocks of 64 tokens) and a run is stored BLOCK-MAJOR:
//          [run][block of 64 dims (the last one zero-padded)][64 tokens][64 dims], so that the attention kernel's
//          [64 tokens x 64 dims] boxes are 8 KiB of contiguous memory (boxes that take 128 bytes out of every
//          1152-byte token row stream from HBM at 4.6 TB/s, contiguous ones at 7.0 TB/s).
struct MlaCache {
  __half *pool;
  const int *block_table;    // [n_slots][max_blocks]
  int max_blocks, n_slots;
  long long pool_blocks;
  int run;                   // 1 or 4
};
// Halfs per cached token in the pool (run = 4: whole blocks of 64 dims).
inline long long mla_token_halfs(int row_halfs, int run) { return run == 1 ? row_halfs : (long long)((row_halfs + 63) / 64) * 64; }
#ifdef __CUDACC__
// Where value e of the token at offset `off` of page `blk` lives.
__device__ __forceinline__ __half *mla_cache_at(const MlaCache &c, int row_halfs, int blk, int off, int e) {
  if (c.run == 1) return c.pool + ((size_t)blk * KV_BLOCK + off) * row_halfs + e;
  const int nblk = (row_halfs + 63) >> 6, r = blk >> 2, tok = (blk & 3) * KV_BLOCK + off;
  return c.pool + (((size_t)r * nblk + (e >> 6)) * 64 + tok) * 64 + (e & 63);
}
#endif

// Rows of the head-major activation matrices ([head][rows_per_head][K]) for a program of BN padded rows: the
// grouped GEMMs take blocks of at most 64 rows.
inline int mla_group_rows(int BN) { return BN <= 64 ? BN : 64; }
inline int mla_rows_per_head(int BN) { return (BN + mla_group_rows(BN) - 1) / mla_group_rows(BN) * mla_group_rows(BN); }

// From the q / kv_a projection of a row (columns: nh x [nope | rope], then rank + rope):
//   latent = RMSNorm(kv_a[:rank]) * gains and the rotated rotary key -> the row's cache position (fp16; padding
//   rows write nothing);  q_nope -> bf16 hi/lo, head-major [nh][rows_per_head][nope];  rotated q_rope -> fp32
//   [R][nh][rope].  rope_tab: (cos, sin) [position][rope / 2].
cudaError_t launch_mla_post(const GemmOut &qkv, const Rows &rows, const float2 *rope_tab, const MlaDims &d,
                            const __nv_bfloat16 *kv_gains, float eps, const MlaCache &cache, int rows_per_head,
                            __nv_bfloat16 *qn_hi, __nv_bfloat16 *qn_lo, float *q_rope, int *d_status, cudaStream_t st);

// Tensor maps over one layer's latent pages for the attention kernel.
// page_run: pool pages per TMA box (1, or 4 where every row's block table holds its pages in aligned runs of four
// consecutive pool pages: launch_mla_attention takes the same value)
int mla_encode_maps(CUtensorMap *tmC, CUtensorMap *tmV, const void *pool, long long pool_pages, int rank, int rope, int page_run);
// Floats of the partial results for R rows of at most max_context cached tokens: (max, sum) pairs, then outputs.
long long mla_part_ml_floats(int R, int nh, int max_context);
long long mla_part_o_floats(int R, int nh, int rank, int max_context);
int mla_max_splits(int max_context);

// Absorbed attention of every row over its cached tokens.  q_lat element (r, h, d) sits at
// q_lat[r * q_row_stride + h * q_head_stride + d]; q_rope is [R][nh][rope].  A row's cached-token count is
// ctx[r] (rows == nullptr; its block-table row is r) or rows->active[r] ? rows->pos[r] + 1 : 0 (its block-table
// row is rows->slot[r]).  The result goes to o_lat (fp32 [R][nh][rank]) or, when o_lat is null, to the bf16 hi/lo
// pair out_hi / out_lo laid out head-major [nh][rows_per_head][rank]; rows without cached tokens keep what they held.
cudaError_t launch_mla_attention(const CUtensorMap &tmC, const CUtensorMap &tmV, const float *q_lat, long long q_row_stride,
                                 long long q_head_stride, const float *q_rope, const int *block_table, int max_blocks,
                                 const int *ctx, const Rows *rows, int R, const MlaDims &d, float scale, int max_splits,
                                 float2 *part_ml, float *part_o, float *o_lat, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                 int rows_per_head, int num_sms, int *d_status, bool pdl, cudaStream_t st, int page_run);

// The value part of the grouped up-projection result uv [nh * rows_per_head][nope + vh] (columns nope.. of every
// row) -> bf16 hi/lo [R][nh * vh], the o-projection's activations.
cudaError_t launch_mla_ao_split(const float *uv, int R, int rows_per_head, const MlaDims &d, __nv_bfloat16 *ao_hi,
                                __nv_bfloat16 *ao_lo, cudaStream_t st);
// out [nh * rank][nope] = the transposed key up-projections: out[h * rank + c][i] = wkv_b[(h * (nope + vh) + i) * rank + c].
cudaError_t launch_mla_transpose_uk(const __nv_bfloat16 *wkv_b, const MlaDims &d, __nv_bfloat16 *out, cudaStream_t st);
// (bench set-up) fills cached positions [0, n) of a slot in one layer with seeded N(0, std^2) values.
cudaError_t launch_mla_fill(const MlaCache &cache, int row_halfs, int layer, int slot, int n, float std, uint64_t seed, cudaStream_t st);
// (debug) cached rows [pos0, pos0 + n) of a slot <-> fp32 [n][rank + rope].
cudaError_t launch_mla_copy(const MlaCache &cache, int row_halfs, int slot, int pos0, int n, float *buf, int write, cudaStream_t st);

}  // namespace corun
