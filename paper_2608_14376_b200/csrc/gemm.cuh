// Decode / prefill-chunk GEMM  out[r, n] = sum_k W[n, k] * (Xhi[r, k] + Xlo[r, k]).
//
// The weight matrix is the 128-row MMA operand, the (padded) rows of
// activations are the N operand, so one fixed tiling serves every row count
// up to 256.  The flat space of (weight tile, 64-wide k-block) pairs is cut
// into one contiguous, equally sized range per CTA; the cut depends on the
// shape (N, K) and the grid only, never on which rows are occupied.  A tile
// whose k-blocks all belong to one CTA is written straight to `direct`;
// otherwise each CTA writes a partial to its workspace slot and the consumer
// adds the partials in ascending CTA order (gemm_load).  No atomics anywhere.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace corun {

// Last CUDA runtime error (cudaError_t), or 100000 + CUresult for driver calls.
extern int g_last_cuda_error;

constexpr int GEMM_TILE_M = 128;   // weight rows per tile
constexpr int GEMM_BLOCK_K = 64;   // bf16 elements per k-block (= one 128-byte swizzle row)
constexpr int GEMM_THREADS = 192;  // warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue

// What a consumer kernel needs to read a GEMM result.
struct GemmOut {
  const float *direct;   // [rows, N]; valid for tiles owned by one CTA
  const float *ws;       // [(cta*2 + slot), BN, 128] partials
  const int *cta_start;  // [grid + 1] first flat k-block of each CTA
  const int *tile_cbeg;  // [n_tiles] first CTA touching the tile
  const int *tile_cend;  // [n_tiles] last CTA touching the tile
  int N, KB, BN;
};

// Value (r, n) of a GEMM result, partials added in ascending CTA order.
__device__ __forceinline__ float gemm_load(const GemmOut &g, int r, int n) {
  const int t = n >> 7, row = n & 127;
  const int c0 = g.tile_cbeg[t], c1 = g.tile_cend[t];
  if (c0 == c1) return g.direct[(size_t)r * g.N + n];
  float acc = 0.f;
  const int first_kb = t * g.KB;
  for (int c = c0; c <= c1; ++c) {
    const int slot = (g.cta_start[c] >= first_kb) ? 0 : 1;
    acc += g.ws[((size_t)(c * 2 + slot) * g.BN + r) * 128 + row];
  }
  return acc;
}

// Static launch description of one GEMM shape (built once at init).
struct GemmPlan {
  CUtensorMap tmW, tmHi, tmLo;
  int N = 0, K = 0, R = 0, BN = 0;   // weight rows, reduction length, real rows, padded rows
  int n_tiles = 0, KB = 0, grid = 0, stages = 0, tmem_cols = 0;
  uint32_t idesc = 0;
  size_t smem_bytes = 0;
  float *direct = nullptr;           // not owned
  float *ws = nullptr;               // not owned
  int *d_cta_start = nullptr, *d_tile_cbeg = nullptr, *d_tile_cend = nullptr;  // owned (one allocation)
  int *d_split_tiles = nullptr;      // tiles with partials (same allocation)
  int n_split_tiles = 0;
  GemmOut out() const { return GemmOut{direct, ws, d_cta_start, d_tile_cbeg, d_tile_cend, N, KB, BN}; }
};

// Workspace floats needed by any plan with this grid and BN.
inline size_t gemm_ws_floats(int grid, int BN) { return (size_t)grid * 2 * BN * 128; }

// Builds the plan: tensor maps for W [N, K] bf16 and the split activations
// Xhi / Xlo [BN, K] bf16 (row pitch K), the CTA partition and its tables.
// Returns 0 or a negative corun_status.
int gemm_plan_create(GemmPlan *p, const void *W, int N, int K, const void *Xhi, const void *Xlo, int R, int BN,
                     float *direct, float *ws, int num_sms);
void gemm_plan_destroy(GemmPlan *p);
// Enqueues the GEMM.  `W` may override the weight matrix of the plan (same
// shape) by passing a different tensor map.
cudaError_t gemm_launch(const GemmPlan &p, const CUtensorMap *tmW_override, int *d_status, cudaStream_t st);
// Encodes a tensor map for a bf16 [rows, K] row-major matrix with a [box_rows, 64] box, 128-byte swizzle.
int gemm_encode_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows);
// Opts the GEMM kernel into its dynamic shared-memory size (idempotent, allocates nothing).
cudaError_t gemm_prepare_kernel();
// direct[r, n] = gemm_load(r, n) for every tile that has partials (makes `direct` a plain matrix).
cudaError_t gemm_fixup_launch(const GemmPlan &p, cudaStream_t st);

}  // namespace corun
