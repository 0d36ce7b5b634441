// Decode / prefill-chunk GEMM  out[r, n] = sum_k W[n, k] * (Xhi[r, k] + Xlo[r, k]).
//
// The rows of activations (up to 256, in blocks of 128) are the M operand of
// the MMA and a tile of 256 weight rows is its N operand, so every tcgen05.mma
// is a full-size 128 x 256 x 16 instruction whatever the row count; one fixed
// tiling serves every row count.  The flat space of (weight tile, 64-wide k-block) pairs is cut
// into one contiguous, equally sized range per CTA; the cut depends on the
// shape (N, K) and the grid only, never on which rows are occupied.  A tile
// whose k-blocks all belong to one CTA is written straight to `direct`;
// otherwise each CTA writes a partial to its workspace slot and the consumer
// adds the partials in ascending CTA order (gemm_load).  No atomics anywhere.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace corun {

// Last CUDA runtime error (cudaError_t), or 100000 + CUresult for driver calls.
extern int g_last_cuda_error;

constexpr int GEMM_TILE_N = 256;   // weight rows per tile (the MMA's N)
constexpr int GEMM_ROW_BLOCK = 128; // activation rows per MMA (the MMA's M)
constexpr int GEMM_BLOCK_K = 64;   // bf16 elements per k-block (= one 128-byte swizzle row)
constexpr int GEMM_THREADS = 192;  // warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue

// What a consumer kernel needs to read a GEMM result.
struct GemmOut {
  const float *direct;   // [rows, N]; valid for tiles owned by one CTA
  const float *ws;       // [(cta*2 + slot), BN, 256] partials
  const int *tile_first; // [n_tiles] 2 * (first CTA touching the tile) + (the slot that CTA used for it)
  const int *tile_cend;  // [n_tiles] last CTA touching the tile (every later CTA used slot 0)
  int N, KB, BN;
};

// Value (r, n) of a GEMM result, partials added in ascending CTA order.
__device__ __forceinline__ float gemm_load(const GemmOut &g, int r, int n) {
  const int t = n / GEMM_TILE_N, col = n % GEMM_TILE_N;
  const int f = g.tile_first[t], c0 = f >> 1, c1 = g.tile_cend[t];
  if (c0 == c1) return g.direct[(size_t)r * g.N + n];
  const float *p = g.ws + ((size_t)r) * GEMM_TILE_N + col;
  const size_t cta_stride = (size_t)2 * g.BN * GEMM_TILE_N;
  float acc = 0.f;
  acc += p[(size_t)f * g.BN * GEMM_TILE_N];
  for (int c = c0 + 1; c <= c1; ++c) acc += p[(size_t)c * cta_stride];
  return acc;
}

// Four consecutive values (n % 4 == 0, N % 4 == 0) with the same summation order as gemm_load.
// Loads are issued four partials at a time; an absent partial contributes +0.0f.
__device__ __forceinline__ float4 gemm_load4(const GemmOut &g, int r, int n) {
  const int t = n / GEMM_TILE_N, col = n % GEMM_TILE_N;
  const int f = g.tile_first[t], c0 = f >> 1, c1 = g.tile_cend[t];
  if (c0 == c1) return *reinterpret_cast<const float4 *>(g.direct + (size_t)r * g.N + n);
  const float *p = g.ws + ((size_t)r) * GEMM_TILE_N + col;
  const size_t cta_stride = (size_t)2 * g.BN * GEMM_TILE_N;
  float4 acc = *reinterpret_cast<const float4 *>(p + (size_t)f * g.BN * GEMM_TILE_N);
  acc.x += 0.f; acc.y += 0.f; acc.z += 0.f; acc.w += 0.f;   // same rounding path as 0 + first partial
  for (int c = c0 + 1; c <= c1; c += 4) {
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      v[j] = (c + j <= c1) ? *reinterpret_cast<const float4 *>(p + (size_t)(c + j) * cta_stride)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w;
    }
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
  int *d_cta_start = nullptr, *d_tile_first = nullptr, *d_tile_cend = nullptr;  // owned (one allocation)
  int *d_split_tiles = nullptr;      // tiles with partials (same allocation)
  int n_split_tiles = 0;
  // Optional store mask (device, not owned): row r of weight tile t is stored only if
  // row_keep[r * keep_pitch + t / keep_div] != 0 (rows that no consumer will read are skipped).
  const float *row_keep = nullptr;
  int keep_pitch = 0, keep_div = 1;
  // Grouped mode (gemm_plan_create_grouped): the CTAs take the (group, weight tile) pairs in turn; see gemm.cu.
  const int *group_tab = nullptr;    // device, not owned: per group (first weight row, first weight k-block, rows),
                                     // then ONE more int: the number of groups in use (the first ones);
                                     // keep_div = -1 tells the kernel that no kernel of the same stream writes it
  int tiles_per_group = 0;
  // Gate / up GEMM with SwiGLU in the epilogue (gemm_plan_create_swiglu): the bf16 hi/lo output [BN, N / 2].
  __nv_bfloat16 *sw_hi = nullptr, *sw_lo = nullptr;
  int sw_half = 0;                   // gate rows (= up rows) per tile
  // Above 64 padded rows the rows form two blocks (65..128 rows: stacked blocks of 64 rows; above: row blocks of 128
  // rows).  Device int, not owned, written by an earlier kernel of the step: bit b set = block b holds a request
  // this step; null = both blocks.  An absent block is neither loaded nor multiplied nor stored.
  const int *row_blocks = nullptr;
  GemmOut out() const { return GemmOut{direct, ws, d_tile_first, d_tile_cend, N, KB, BN}; }
};

// Workspace floats needed by any plan with this grid and BN.
inline size_t gemm_ws_floats(int grid, int BN) { return (size_t)grid * 2 * BN * GEMM_TILE_N; }

// Builds the plan: tensor maps for W [N, K] bf16 and the split activations
// Xhi / Xlo [BN, K] bf16 (row pitch K), the CTA partition and its tables.
// Returns 0 or a negative corun_status.
int gemm_plan_create(GemmPlan *p, const void *W, int N, int K, const void *Xhi, const void *Xlo, int R, int BN,
                     float *direct, float *ws, int num_sms);
void gemm_plan_destroy(GemmPlan *p);
// Grouped GEMM over at most n_groups groups of up to BN <= 64 rows each: group g multiplies rows g * BN .. of
// Xhi / Xlo ([n_groups * BN, K]) with N weight rows starting at the row, and K elements starting at the k-block,
// that group_tab names for it, into rows g * BN .. of `direct` ([n_groups * BN, N]).  W is [w_rows, w_cols]
// bf16.  group_tab has 3 * n_groups + 1 ints: the last one is the number of groups in use (groups 0 .. that - 1).
// At most num_sms CTAs take the (group, tile of 256 weight rows) pairs of the groups in use in turn, all k-blocks
// of a tile: no partials.  N % 256 == 0.
int gemm_plan_create_grouped(GemmPlan *p, const void *W, long long w_rows, int w_cols, int N, int K, const void *Xhi,
                             const void *Xlo, int n_groups, int BN, float *direct, const int *group_tab, int num_sms);
// The same for gate / up matrices ([2F, K] per group: F gate rows, then F up rows, from the group's first weight row)
// with the SwiGLU in the epilogue: row_scale[g * BN + r] * silu(gate) * up as a bf16 hi/lo pair [n_groups * BN, F].
// Tiles of `half` gate rows and the `half` up rows of the same outputs (F % half == 0, 64 <= half <= 128).
int gemm_plan_create_grouped_swiglu(GemmPlan *p, const void *W, long long w_rows, int F, int K, int half, const void *Xhi,
                                    const void *Xlo, int n_groups, int BN, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                    const float *row_scale, const int *group_tab, int num_sms);
// Gate / up GEMM with the SwiGLU in its epilogue: W is [2F, K] (F gate rows, then F up rows; F % 8 == 0);
// out_hi / out_lo [BN, F] receive silu(gate) * up of rows 0 .. R-1 as a bf16 hi/lo pair.  A tile is
// gemm_swiglu_half(F, num_sms) gate rows with the up rows of the same outputs, and every CTA owns whole tiles
// (one each when the SMs allow), so there are no partials; a tensor map that overrides the plan's at launch
// must have a box of that many rows (gemm_encode_map(.., box_rows = gemm_swiglu_half(..))).
int gemm_swiglu_half(int F, int num_sms);
int gemm_plan_create_swiglu(GemmPlan *p, const void *W, int F, int K, const void *Xhi, const void *Xlo, int R, int BN,
                            __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int num_sms);
// The same for a stack of n_blocks gate / up matrices (the experts of a Mixture-of-Experts layer): W is
// [n_blocks * 2 * Fb, K], block e = Fb gate rows then Fb up rows; out_hi / out_lo [BN, n_blocks * Fb] receive
// row_scale[r * n_blocks + e] * silu(gate) * up in columns e * Fb .., exact zeros where the scale is zero (the
// row did not select the expert).  A tile is gemm_swiglu_blocks_half(Fb, n_blocks, num_sms) gate rows of one
// block with their up rows (0: no multiple of 8 in 64..128 divides Fb); whole tiles, no partials.
int gemm_swiglu_blocks_half(int Fb, int n_blocks, int num_sms);
int gemm_plan_create_swiglu_blocks(GemmPlan *p, const void *W, int n_blocks, int Fb, int K, const void *Xhi, const void *Xlo,
                                   int R, int BN, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, const float *row_scale,
                                   int num_sms);
// The allocation-free half of gemm_plan_create: fills every host-side field and tensor map of the
// plan and writes the partition tables (cta_start, tile_first, tile_cend, split_tiles) to `tab`
// (capacity tab_cap ints; *tab_ints = ints used).  gemm_plan_bind_tables points the plan at a device
// copy of those tables.
int gemm_plan_fill(GemmPlan *p, const void *W, int N, int K, const void *Xhi, const void *Xlo, int R, int BN,
                   float *direct, float *ws, int num_sms, int *tab, int tab_cap, int *tab_ints);
void gemm_plan_bind_tables(GemmPlan *p, int *d_tab);
// Enqueues the GEMM.  `W` may override the weight matrix of the plan (same
// shape) by passing a different tensor map.
cudaError_t gemm_launch(const GemmPlan &p, const CUtensorMap *tmW_override, int *d_status, cudaStream_t st,
                        unsigned long long *trace = nullptr,   // optional [grid][8] globaltimer stamps (debug)
                        bool pdl = false);                     // programmatic dependent launch (row program)
// Encodes a tensor map for a bf16 [rows, K] row-major matrix with a [box_rows, 64] box, 128-byte swizzle.
int gemm_encode_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows);
// Opts the GEMM kernel into its dynamic shared-memory size (idempotent, allocates nothing).
cudaError_t gemm_prepare_kernel();
// Tensor map for a 16-bit [rows, cols] row-major matrix with a [box_rows, box_cols] box: 64 columns
// (128 bytes, 128-byte swizzle) or 16 columns (32 bytes, 32-byte swizzle).
int tma_encode_2d(CUtensorMap *m, const void *base, int is_fp16, unsigned long long rows, int cols, int box_rows,
                  int box_cols);
// Tensor map over fp16 data seen as a 4-dimensional array: dims[0] elements are contiguous, strides[i] is the byte
// distance between consecutive indices of dimension i + 1 (a multiple of 16; they need not ascend); the box's
// innermost extent is 64 elements (128 bytes, 128-byte swizzle).  The box lands in shared memory densely,
// dimension 0 fastest.
int tma_encode_fp16_4d(CUtensorMap *m, const void *base, const unsigned long long dims[4], const unsigned long long strides[3],
                       const unsigned box[4]);
// The same with 2 to 5 dimensions (dims / box: nd values, strides: nd - 1 byte strides of dimensions 1 ..).
int tma_encode_fp16_nd(CUtensorMap *m, const void *base, int nd, const unsigned long long *dims, const unsigned long long *strides,
                       const unsigned *box);
// direct[r, n] = gemm_load(r, n) for every tile that has partials (makes `direct` a plain matrix).
cudaError_t gemm_fixup_launch(const GemmPlan &p, cudaStream_t st, bool pdl = false);

}  // namespace corun
