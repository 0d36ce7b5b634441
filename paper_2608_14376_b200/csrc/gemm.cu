// tcgen05 / TMEM / TMA GEMM for sm_100a with a static, shape-keyed work partition.
#include "gemm.cuh"

#include <cudaTypedefs.h>

#include <cstdlib>
#include <vector>

#include "../../include/corun.h"
#include "launch.cuh"
#include "ptx.cuh"

namespace corun {

int g_last_cuda_error = 0;
bool g_use_pdl = !(getenv("CORUN_NO_PDL") && atoi(getenv("CORUN_NO_PDL")) != 0);

namespace {

constexpr int MAX_STAGES = 8;
constexpr int GEMM_MAX_DYN_SMEM = 209 * 1024;   // leaves room for the static shared memory within the 227 KiB of a CTA
constexpr uint32_t W_TILE_BYTES = GEMM_TILE_N * GEMM_BLOCK_K * 2;          // 32 KiB
constexpr uint32_t A_BLOCK_BYTES = GEMM_ROW_BLOCK * GEMM_BLOCK_K * 2;      // 16 KiB: what one MMA reads of A

// Role loops walk the CTA's flat k-block range [k0, k1) segment by segment; a
// segment is the part of the range that falls into one weight tile.
//
// Operands: A = activations (hi or lo), 128 rows per MMA, K-major, 128-byte
// swizzle; B = 256 weight rows, same layout; D = fp32 [128 rows x 256 weight
// rows] in TMEM (lane = activation row, column = weight row), one accumulator
// per block of 128 activation rows.  When fewer than 128 rows are loaded the
// MMA still reads 128 rows of shared memory; the extra accumulator lanes hold
// meaningless values that are never read back.
// MASKED: the optional store mask of the epilogue (a separate instantiation, so that the plain kernel is
// exactly the code it was without it).
// GROUPED (with STACKED): a tile is one whole output tile of one group (an expert's rows, gathered into blocks
// of BN rows).  group_tab holds, per group, the first weight row, the first weight k-block and the number of
// rows, and behind its keep_pitch entries the number of groups in use (the first ones); the CTAs take the tiles
// of those groups in turn (tile cta, cta + grid, ...), streaming from one tile into the next like the plain
// kernel.  The group's activations are rows group * BN .. of the activation matrices, its output rows
// group * BN .. of `direct` (N columns wide, tiles_per_group tiles).
// SWIGLU: W is a gate / up matrix ([2F, K]: F gate rows, then F up rows).  A tile is sw_half gate rows and the
// sw_half up rows of the same outputs (two boxes of sw_half rows land in one stage; the MMA's N is 2 * sw_half),
// every CTA owns whole tiles, and the epilogue writes silu(gate) * up as a bf16 hi/lo pair ([BN, F]) instead of
// fp32 sums: no partials, no separate SwiGLU kernel.  tmW then has a box of sw_half rows.
// SWIGLU with GROUPED: a group's N weight rows are one gate / up matrix (N / 2 gate rows, then N / 2 up rows) starting at
// the group's first weight row; row_keep holds one factor per output row (the routing weight of the gathered row) and
// the epilogue writes factor * silu(gate) * up to rows group * BN .. of the bf16 hi/lo output ([groups * BN, N / 2]).
// SWIGLU with MASKED: W is a stack of keep_pitch such matrices (the experts of a Mixture-of-Experts layer: block e =
// Fb gate rows, then Fb up rows, Fb = N / (2 * keep_pitch)), a tile belongs to one block (keep_div tiles per block),
// and the epilogue writes row_keep[r, e] * silu(gate) * up, exact zeros where row r did not select block e, to
// columns e * Fb .. of the bf16 hi/lo output [BN, N / 2].
// NSB = 2 (with STACKED; 65..128 padded rows): TWO stacked blocks of 64 rows, each with its own 128-row A tile (hi rows
// 0-63, lo rows 64-127) and its own accumulator.  *row_blocks (bit b: rows 64 b .. hold active rows; written by an
// earlier kernel of the step, or null = both) says which blocks exist this step: an absent block is neither loaded
// nor multiplied nor stored (its output rows keep what they held: nobody reads rows without a request).  A row's
// value does not depend on which blocks exist.
template <bool MASKED, bool STACKED, bool GROUPED, bool SWIGLU, int NSB = 1>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_streamk_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmHi,
                    const __grid_constant__ CUtensorMap tmLo, float *__restrict__ direct, float *__restrict__ ws,
                    const int *__restrict__ cta_start, int N, int KB, int BN, int R, int stages, int tmem_cols,
                    uint32_t idesc, const float *row_keep, int keep_pitch, int keep_div, const int *group_tab,
                    int tiles_per_group, int *status, unsigned long long *trace, __nv_bfloat16 *__restrict__ sw_hi,
                    __nv_bfloat16 *__restrict__ sw_lo, int sw_half, const int *row_blocks) {
  extern __shared__ uint8_t smem_raw[];
  // optional per-CTA timeline (debug): 8 globaltimer stamps
#define TRACE(i) do { if (trace) trace[(size_t)blockIdx.x * 8 + (i)] = globaltimer_ns(); } while (0)
  if (threadIdx.x == 0) TRACE(0);
  griddep_launch_dependents();   // the next kernel may start its prologue
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];    // one pair per accumulator buffer
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xch[2][64 * 33];   // stacked epilogue: W*hi and W*lo of 64 rows x 32 columns (row pitch 33: no bank conflicts)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  // GROUPED: the group of the CTA's i-th tile (read only after the wait for the table below): group, tile inside it, first weight row, first weight k-block, rows in use
  int g_tile = -1, g_id = 0, g_j = 0, g_wrow = 0, g_wk = 0, g_rows = 0;
  auto look = [&](int tile) {
    if (GROUPED && tile != g_tile) {
      const int t = cta + tile * (int)gridDim.x;
      g_tile = tile;
      g_id = t / tiles_per_group;
      g_j = t - g_id * tiles_per_group;
      g_wrow = group_tab[3 * g_id];
      g_wk = group_tab[3 * g_id + 1];
      g_rows = group_tab[3 * g_id + 2];
    }
  };
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t x_bytes = (uint32_t)BN * GEMM_BLOCK_K * 2;         // BN * 128 B
  // Up to 64 rows: hi and lo share one 128-row A tile (hi in rows 0.., lo in rows 64..), so one MMA
  // per k-slice yields W*hi in accumulator lanes 0-63 and W*lo in lanes 64-127; the epilogue adds them.
  constexpr bool stacked = STACKED;                 // = (BN <= 64), fixed at compile time
  // not stacked, two row blocks: the hi tiles of both blocks (128 rows each, whatever BN is), then the lo tiles
  const uint32_t x_reg = (!stacked && BN > GEMM_ROW_BLOCK) ? 2u * A_BLOCK_BYTES : x_bytes;
  const uint32_t lo_off = stacked ? (uint32_t)(64 * GEMM_BLOCK_K * 2) : x_reg;
  const uint32_t w_tile_bytes = SWIGLU ? (uint32_t)(2 * sw_half * GEMM_BLOCK_K * 2) : W_TILE_BYTES;
  // SWIGLU: first gate row of a tile, and the distance to the up rows of the same outputs
  const int sw_fb = (SWIGLU && MASKED) ? N / (2 * keep_pitch) : N / 2;
  auto sw_gate_row = [&](int tile) {
    if (GROUPED) return g_wrow + g_j * sw_half;       // (the caller has looked the tile's group up)
    if (SWIGLU && MASKED) {
      const int e = tile / keep_div;
      return e * 2 * sw_fb + (tile - e * keep_div) * sw_half;
    }
    return tile * sw_half;
  };
  const uint32_t stage_bytes = w_tile_bytes + (stacked ? (uint32_t)NSB * A_BLOCK_BYTES : 2 * x_reg);
  uint32_t tx_bytes = w_tile_bytes + 2 * x_bytes;                   // (NSB = 2: set once the blocks are known)
  const int n_rb = NSB == 2 ? 1 : (BN + GEMM_ROW_BLOCK - 1) / GEMM_ROW_BLOCK;   // blocks of 128 activation rows
  // up to 128 rows need 256 TMEM columns: two accumulator buffers fit, so the epilogue of one
  // segment overlaps the MMAs of the next (NSB = 2: only while one block exists, see below)
  int n_acc = (n_rb == 1) ? 2 : 1;
  const uint32_t acc_cols = (uint32_t)n_rb * GEMM_TILE_N;
  // NSB = 2: which blocks exist (read behind the wait for the predecessor), and an accumulator's first column
  // Not STACKED (above 128 padded rows): the blocks are the row blocks of 128 rows (hi and lo boxes of 128 rows each),
  // left out in the same way; with one block left its two accumulator buffers alternate as for up to 128 rows.
  constexpr bool DYN_BLOCKS = NSB == 2 || (!STACKED && !GROUPED);
  int bmask = NSB == 2 ? 3 : (1 << n_rb) - 1;
  auto read_blocks = [&]() {
    if (DYN_BLOCKS) {
      const int all = NSB == 2 ? 3 : (1 << n_rb) - 1;
      if (row_blocks) { griddep_wait(); bmask = *reinterpret_cast<const volatile int *>(row_blocks) & all; }
      if (bmask == 0) bmask = 1;                    // a step without requests: block 0 is computed and ignored
      n_acc = bmask == 3 ? 1 : 2;
      tx_bytes = w_tile_bytes + (uint32_t)__popc(bmask) * (NSB == 2 ? A_BLOCK_BYTES : 2 * (n_rb == 1 ? x_bytes : A_BLOCK_BYTES));
    }
  };
  auto acc_col = [&](int acc, int b) {
    return DYN_BLOCKS ? (uint32_t)(n_acc == 2 ? acc : b) * GEMM_TILE_N : (uint32_t)acc * acc_cols + (STACKED ? 0u : (uint32_t)b * GEMM_TILE_N);
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tmem_full_bar[a]), 1);
      mbar_init(smem_u32(&tmem_empty_bar[a]), 128);
    }
    fence_mbar_init();
    fence_proxy_async();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmHi);
    prefetch_tensormap(&tmLo);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), (uint32_t)tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int *abort_p = &abort_flag;
  if (threadIdx.x == 0) TRACE(1);

  // GROUPED: the CTA walks the tiles cta, cta + grid, ... of the groups in use (their number follows the table's
  // keep_pitch entries), every tile whole; the flat range counts the k-blocks of those tiles.
  int k0, k1;
  if (GROUPED) {
    if (keep_div >= 0) griddep_wait();              // the group table comes from an earlier kernel (keep_div < 0: it is fixed)
    const int used = min(group_tab[3 * keep_pitch], keep_pitch) * tiles_per_group;
    k0 = 0;
    k1 = cta < used ? (used - cta + (int)gridDim.x - 1) / (int)gridDim.x * KB : 0;
  } else {
    k0 = cta_start[cta];
    k1 = cta_start[cta + 1];
  }
  int fail = 0;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      const uint64_t pol_w = l2_policy_evict_first();   // weights are streamed once per step
      const uint64_t pol_x = l2_policy_evict_last();    // activations are re-read by every CTA
      // The weights depend on no earlier kernel: fill the ring with weight tiles first, then wait for
      // the predecessor (which produces the activations) and add the activation tiles to the same
      // barriers.
      const int n_pre = min(stages, k1 - k0);
      for (int it = 0; it < n_pre; ++it) {
        const int g = k0 + it, tile = g / KB, kb = g - tile * KB;
        look(tile);
        const uint32_t fb = smem_u32(&full_bar[it]);
        if (DYN_BLOCKS) mbar_expect_tx(fb, w_tile_bytes);   // the activations' bytes and the arrival follow behind the wait
        else mbar_arrive_expect_tx(fb, tx_bytes);
        if (SWIGLU) {
          tma_load_2d(tiles_base + (uint32_t)it * stage_bytes, &tmW, kb * GEMM_BLOCK_K, sw_gate_row(tile), fb, pol_w);
          tma_load_2d(tiles_base + (uint32_t)it * stage_bytes + w_tile_bytes / 2, &tmW, kb * GEMM_BLOCK_K,
                      sw_gate_row(tile) + sw_fb, fb, pol_w);
        } else
        tma_load_2d(tiles_base + (uint32_t)it * stage_bytes, &tmW, (GROUPED ? g_wk + kb : kb) * GEMM_BLOCK_K,
                    GROUPED ? g_wrow + g_j * GEMM_TILE_N : tile * GEMM_TILE_N, fb, pol_w);
        if (it == 0) TRACE(2);
      }
      griddep_wait();
      read_blocks();
      // the activation tiles of a stage (NSB = 2: a hi and a lo box of 64 rows per block that exists)
      auto load_x = [&](uint32_t dst, int kb, uint32_t fb) {
        if (NSB == 2) {
#pragma unroll
          for (int b = 0; b < 2; ++b)
            if ((bmask >> b) & 1) {
              tma_load_2d(dst + w_tile_bytes + (uint32_t)b * A_BLOCK_BYTES, &tmHi, kb * GEMM_BLOCK_K, 64 * b, fb, pol_x);
              tma_load_2d(dst + w_tile_bytes + (uint32_t)b * A_BLOCK_BYTES + lo_off, &tmLo, kb * GEMM_BLOCK_K, 64 * b, fb, pol_x);
            }
        } else if (DYN_BLOCKS && n_rb == 2) {
#pragma unroll
          for (int b = 0; b < 2; ++b)
            if ((bmask >> b) & 1) {
              tma_load_2d(dst + w_tile_bytes + (uint32_t)b * A_BLOCK_BYTES, &tmHi, kb * GEMM_BLOCK_K, GEMM_ROW_BLOCK * b, fb, pol_x);
              tma_load_2d(dst + w_tile_bytes + lo_off + (uint32_t)b * A_BLOCK_BYTES, &tmLo, kb * GEMM_BLOCK_K, GEMM_ROW_BLOCK * b, fb, pol_x);
            }
        } else {
          tma_load_2d(dst + w_tile_bytes, &tmHi, kb * GEMM_BLOCK_K, GROUPED ? g_id * BN : 0, fb, pol_x);
          tma_load_2d(dst + w_tile_bytes + lo_off, &tmLo, kb * GEMM_BLOCK_K, GROUPED ? g_id * BN : 0, fb, pol_x);
        }
      };
      for (int it = 0; it < n_pre; ++it) {
        const int g = k0 + it, tile = g / KB, kb = g - tile * KB;
        look(tile);
        const uint32_t fb = smem_u32(&full_bar[it]);
        const uint32_t dst = tiles_base + (uint32_t)it * stage_bytes;
        if (DYN_BLOCKS) mbar_arrive_expect_tx(fb, tx_bytes - w_tile_bytes);
        load_x(dst, kb, fb);
      }
      int it = n_pre;
      for (int g = k0 + n_pre; g < k1; ++g, ++it) {
        const int tile = g / KB, kb = g - tile * KB;
        look(tile);
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_p)) { fail = DEV_TIMEOUT_PRODUCER; break; }
        const uint32_t fb = smem_u32(&full_bar[s]);
        const uint32_t dst = tiles_base + (uint32_t)s * stage_bytes;
        mbar_arrive_expect_tx(fb, tx_bytes);
        if (SWIGLU) {
          tma_load_2d(dst, &tmW, kb * GEMM_BLOCK_K, sw_gate_row(tile), fb, pol_w);
          tma_load_2d(dst + w_tile_bytes / 2, &tmW, kb * GEMM_BLOCK_K, sw_gate_row(tile) + sw_fb, fb, pol_w);
        } else
        tma_load_2d(dst, &tmW, (GROUPED ? g_wk + kb : kb) * GEMM_BLOCK_K, GROUPED ? g_wrow + g_j * GEMM_TILE_N : tile * GEMM_TILE_N,
                    fb, pol_w);
        load_x(dst, kb, fb);
      }
      TRACE(3);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      read_blocks();
      int it = 0, seg = 0;
      for (int g = k0; g < k1 && !fail; ++seg) {
        const int tile = g / KB, kb_begin = g - tile * KB;
        const int kb_end = min(KB, kb_begin + (k1 - g));
        const int acc = seg % n_acc;
        const uint32_t use = (uint32_t)(seg / n_acc);     // how often this buffer has been used before
        if (!mbar_wait(smem_u32(&tmem_empty_bar[acc]), (use & 1u) ^ 1u, abort_p)) { fail = DEV_TIMEOUT_MMA; break; }
        tc_fence_after();
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
          const int s = it % stages;
          const uint32_t ph = (uint32_t)(it / stages) & 1u;
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, abort_p)) { fail = DEV_TIMEOUT_MMA; break; }
          if (it == 0) TRACE(4);
          tc_fence_after();
          const uint32_t w_addr = tiles_base + (uint32_t)s * stage_bytes;
          const uint64_t w_desc = umma_desc_sw128(w_addr);
          if (stacked) {
#pragma unroll
            for (int b = 0; b < NSB; ++b) {
              if (NSB == 2 && !((bmask >> b) & 1)) continue;
              const uint64_t a_desc = umma_desc_sw128(w_addr + w_tile_bytes + (uint32_t)b * A_BLOCK_BYTES);
              const uint32_t d_tmem = tmem_base + acc_col(acc, b);
#pragma unroll
              for (int k = 0; k < GEMM_BLOCK_K / 16; ++k) {
                const uint64_t adv = (uint64_t)(k * 2);
                umma_bf16(d_tmem, a_desc + adv, w_desc + adv, idesc, (kb > kb_begin || k > 0) ? 1u : 0u);
              }
            }
          } else {
            for (int rb = 0; rb < n_rb; ++rb) {
              if (DYN_BLOCKS && !((bmask >> rb) & 1)) continue;
              const uint64_t hi_desc = umma_desc_sw128(w_addr + w_tile_bytes + (uint32_t)rb * A_BLOCK_BYTES);
              const uint64_t lo_desc = umma_desc_sw128(w_addr + w_tile_bytes + lo_off + (uint32_t)rb * A_BLOCK_BYTES);
              const uint32_t d_tmem = tmem_base + acc_col(acc, rb);
#pragma unroll
              for (int k = 0; k < GEMM_BLOCK_K / 16; ++k) {
                // advancing 16 bf16 = 32 bytes along K inside the swizzle row: +2 in 16-byte units
                const uint64_t adv = (uint64_t)(k * 2);
                umma_bf16(d_tmem, hi_desc + adv, w_desc + adv, idesc, (kb > kb_begin || k > 0) ? 1u : 0u);
                umma_bf16(d_tmem, lo_desc + adv, w_desc + adv, idesc, 1u);
              }
            }
          }
          umma_commit(smem_u32(&empty_bar[s]));   // frees the stage once these MMAs have read it
        }
        if (fail) break;
        umma_commit(smem_u32(&tmem_full_bar[acc]));    // accumulators of this segment are complete
        g += kb_end - kb_begin;
      }
      TRACE(5);
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int lane_base = (warp & 3) * 32;          // the TMEM lanes this warp may read
    read_blocks();
    int seg = 0;
    for (int g = k0; g < k1; ++seg) {
      const int tile = g / KB, kb_begin = g - tile * KB;
      const int kb_end = min(KB, kb_begin + (k1 - g));
      const bool whole = (kb_begin == 0 && kb_end == KB);
      const int acc = seg % n_acc;
      const uint32_t use = (uint32_t)(seg / n_acc);
      bool ok = mbar_wait(smem_u32(&tmem_full_bar[acc]), use & 1u, abort_p);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { fail = DEV_TIMEOUT_EPILOGUE; break; }
      tc_fence_after();
      if (g + (kb_end - kb_begin) >= k1 && threadIdx.x == 64) TRACE(6);   // last accumulator is ready
      look(tile);
      const int n0 = GROUPED ? g_j * GEMM_TILE_N : tile * GEMM_TILE_N;
      // optional: rows whose entry for this tile's column group is zero are not stored (nobody reads them)
      const float *keep = MASKED ? row_keep + tile / keep_div : nullptr;
      if (SWIGLU) {
        // accumulator columns 0 .. sw_half-1: gate sums of outputs tile * sw_half .., the next sw_half columns: the
        // up sums of the same outputs; every tile is whole
        const int HALF = sw_half;
        // F: outputs per block (the whole matrix unless MASKED); f0: the tile's first output inside its block;
        // o_base: its first column in the output row of N / 2 values; blk: the block (expert) of the tile
        const int blk = MASKED ? tile / keep_div : 0;
        const int F = sw_fb, f0 = (GROUPED ? g_j : MASKED ? tile - blk * keep_div : tile) * HALF;
        const int o_pitch = N / 2, o_base = blk * F + f0;
        // GROUPED: the group's rows in use, its first output row, and row_keep = one weight per output row
        const int sw_rows = GROUPED ? g_rows : R, sw_row0 = GROUPED ? g_id * BN : 0;
        auto silu_mul = [](float gt, float up) { return __fdividef(gt, 1.f + __expf(-gt)) * up; };
        if (stacked) {
         for (int b = 0; b < NSB; ++b) {                // the stacked blocks of 64 rows (one unless NSB = 2)
          if (NSB == 2 && !((bmask >> b) & 1)) continue;
          const int rb0 = 64 * b, rows_b = sw_rows - rb0;   // the block's first row, its rows in use
          const bool lo_warp = lane_base >= 64;
          const int row = (lane_base & 63) + lane;
          const bool warp_needed = (lane_base & 63) < rows_b;   // warp-uniform
          float *xs = xch[lo_warp ? 1 : 0] + row * 33;
          const int te = (int)threadIdx.x - 64, srow = te >> 3, scol = (te & 7) * 4;
          for (int c0 = 0; c0 < HALF; c0 += 32) {
            if (f0 + c0 >= F) break;                   // outputs beyond the matrix (last tile); uniform
            float gt[4][4];
#pragma unroll
            for (int part = 0; part < 2; ++part) {     // 0: the gate columns, 1: the up columns
              if (warp_needed) {
                uint32_t v[32];
                const uint32_t ta = tmem_base + ((uint32_t)lane_base << 16) + acc_col(acc, b) +
                                    (uint32_t)(part * HALF + c0);
                tmem_ld16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                tmem_ld16(ta + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) xs[j] = __uint_as_float(v[j]);
              }
              asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int r = i * 16 + srow;
                if (r < rows_b) {
                  const float *h = xch[0] + r * 33 + scol, *l = xch[1] + r * 33 + scol;
                  const float s0 = h[0] + l[0], s1 = h[1] + l[1], s2 = h[2] + l[2], s3 = h[3] + l[3];
                  if (part == 0) {
                    gt[i][0] = s0; gt[i][1] = s1; gt[i][2] = s2; gt[i][3] = s3;
                  } else if (c0 + scol < HALF && f0 + c0 + scol < F) {   // HALF % 4 == 0, F % 4 == 0
                    float y[4] = {silu_mul(gt[i][0], s0), silu_mul(gt[i][1], s1), silu_mul(gt[i][2], s2),
                                  silu_mul(gt[i][3], s3)};
                    if (MASKED || GROUPED) {           // the row's routing weight for this expert; 0: not selected
                      const float wgt = GROUPED ? row_keep[sw_row0 + r] : row_keep[(size_t)(rb0 + r) * keep_pitch + blk];
#pragma unroll
                      for (int q = 0; q < 4; ++q) y[q] = wgt != 0.f ? wgt * y[q] : 0.f;
                    }
                    __nv_bfloat16 a[4], b2[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                      a[q] = __float2bfloat16_rn(y[q]);
                      b2[q] = __float2bfloat16_rn(y[q] - __bfloat162float(a[q]));
                    }
                    const size_t o = (size_t)(sw_row0 + rb0 + r) * o_pitch + o_base + c0 + scol;
                    *reinterpret_cast<uint2 *>(sw_hi + o) = *reinterpret_cast<const uint2 *>(a);
                    *reinterpret_cast<uint2 *>(sw_lo + o) = *reinterpret_cast<const uint2 *>(b2);
                  }
                }
              }
              asm volatile("bar.sync 1, 128;" ::: "memory");
            }
          }
         }
        } else {
          for (int rb = 0; rb < n_rb; ++rb) {
            if (DYN_BLOCKS && !((bmask >> rb) & 1)) continue;
            const int row_base = rb * GEMM_ROW_BLOCK + lane_base;
            if (row_base >= R) continue;                 // warp-uniform
            const int row = row_base + lane;
            for (int c0 = 0; c0 < HALF; c0 += 8) {
              if (f0 + c0 >= F) break;                   // F % 8 == 0
              uint32_t vg[8], vu[8];
              const uint32_t ta = tmem_base + ((uint32_t)lane_base << 16) + acc_col(acc, rb) + (uint32_t)c0;
              tmem_ld8(ta, vg);
              tmem_ld8(ta + HALF, vu);
              tmem_ld_wait();
              if (row >= R) continue;
              const float wgt = MASKED ? row_keep[(size_t)row * keep_pitch + blk] : 1.f;
              __nv_bfloat16 a[8], b[8];
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                float y = silu_mul(__uint_as_float(vg[q]), __uint_as_float(vu[q]));
                if (MASKED) y = wgt != 0.f ? wgt * y : 0.f;
                a[q] = __float2bfloat16_rn(y);
                b[q] = __float2bfloat16_rn(y - __bfloat162float(a[q]));
              }
              const size_t o = (size_t)row * o_pitch + o_base + c0;
              *reinterpret_cast<uint4 *>(sw_hi + o) = *reinterpret_cast<const uint4 *>(a);
              *reinterpret_cast<uint4 *>(sw_lo + o) = *reinterpret_cast<const uint4 *>(b);
            }
          }
        }
      } else
      if (stacked) {
       for (int b = 0; b < NSB; ++b) {                  // the stacked blocks of 64 rows (one unless NSB = 2)
        if (NSB == 2 && !((bmask >> b) & 1)) continue;
        const int rb0 = 64 * b;                         // the block's first row
        // lanes 0-63 (warps with lane_base 0, 32) hold W*hi of rows 0-63, lanes 64-127 hold W*lo of the
        // same rows: every warp parks 32 columns of its rows in shared memory, then the 128 threads add
        // the two halves and store whole 128-byte row segments (four rows per warp instruction)
        const bool lo_warp = lane_base >= 64;
        const int row = (lane_base & 63) + lane;
        const int rows_valid = (GROUPED ? g_rows : (whole ? R : BN)) - rb0;
        const bool warp_needed = (lane_base & 63) < rows_valid;   // warp-uniform
        float *xs = xch[lo_warp ? 1 : 0] + row * 33;
        const int te = (int)threadIdx.x - 64, srow = te >> 3, scol = (te & 7) * 4;
        const size_t pitch = whole ? (size_t)N : (size_t)GEMM_TILE_N;
        float *dst0 = (GROUPED ? direct + (size_t)g_id * BN * N + n0
                               : (whole ? direct + n0 : ws + (size_t)(cta * 2 + (seg == 0 ? 0 : 1)) * BN * GEMM_TILE_N)) +
                      (size_t)rb0 * pitch;
        const bool vec_ok = whole ? ((N & 3) == 0) : true;
        bool row_on[4];                               // which of this thread's four rows are stored at all
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = i * 16 + srow;
          row_on[i] = r < rows_valid && (!MASKED || rb0 + r >= R || keep[(size_t)(rb0 + r) * keep_pitch] != 0.f);
        }
        for (int c0 = 0; c0 < GEMM_TILE_N; c0 += 32) {
          if (whole && n0 + c0 >= N) break;          // columns beyond the matrix (last tile); uniform
          if (warp_needed) {
            uint32_t v[32];
            const uint32_t ta = tmem_base + ((uint32_t)lane_base << 16) + acc_col(acc, b) + (uint32_t)c0;
            tmem_ld16(ta, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
            tmem_ld16(ta + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) xs[j] = __uint_as_float(v[j]);
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int r = i * 16 + srow;
            if (row_on[i]) {
              const float *h = xch[0] + r * 33 + scol, *l = xch[1] + r * 33 + scol;
              const float4 f = make_float4(h[0] + l[0], h[1] + l[1], h[2] + l[2], h[3] + l[3]);
              float *d = dst0 + (size_t)r * pitch + c0 + scol;
              if (vec_ok && (!whole || n0 + c0 + scol + 4 <= N)) {
                *reinterpret_cast<float4 *>(d) = f;
              } else {
                const int nn = n0 + c0 + scol;
                if (nn < N) d[0] = f.x;
                if (nn + 1 < N) d[1] = f.y;
                if (nn + 2 < N) d[2] = f.z;
                if (nn + 3 < N) d[3] = f.w;
              }
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
       }
      } else
      for (int rb = 0; rb < n_rb; ++rb) {
        if (DYN_BLOCKS && !((bmask >> rb) & 1)) continue;
        const int row_base = rb * GEMM_ROW_BLOCK + lane_base;
        const int rows_valid = whole ? R : BN;      // partials keep the padded row count
        if (row_base >= rows_valid) continue;        // warp-uniform: nothing of this warp's lanes is needed
        const int row = row_base + lane;
        const bool row_ok = row < rows_valid && (!MASKED || row >= R || keep[(size_t)row * keep_pitch] != 0.f);
        float *dst = whole ? direct + (size_t)row * N + n0
                           : ws + ((size_t)(cta * 2 + (seg == 0 ? 0 : 1)) * BN + row) * GEMM_TILE_N;
        const bool vec_ok = whole ? ((N & 3) == 0) : true;
        for (int c0 = 0; c0 < GEMM_TILE_N; c0 += 16) {
          if (whole && n0 + c0 >= N) break;          // columns beyond the matrix (last tile)
          uint32_t v[16];
          tmem_ld16(tmem_base + ((uint32_t)lane_base << 16) + acc_col(acc, rb) + (uint32_t)c0, v);
          tmem_ld_wait();
          if (!row_ok) continue;
          if (vec_ok && (!whole || n0 + c0 + 16 <= N)) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              *reinterpret_cast<float4 *>(dst + c0 + j) =
                  make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                              __uint_as_float(v[j + 3]));
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (n0 + c0 + j < N) dst[c0 + j] = __uint_as_float(v[j]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&tmem_empty_bar[acc]));
      g += kb_end - kb_begin;
    }
    if (threadIdx.x == 64) TRACE(7);
  }

  if (fail) {
    atomicCAS(status, 0, fail);
    // let copies that are still in flight land before the shared memory is given back
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)tmem_cols);
}

__global__ void __launch_bounds__(GEMM_TILE_N) gemm_fixup_kernel(GemmOut g, float *direct, const int *split_tiles) {
  griddep_launch_dependents();
  griddep_wait();
  const int t = split_tiles[blockIdx.x], r = blockIdx.y;
  const int n = t * GEMM_TILE_N + threadIdx.x;
  if (n < g.N) direct[(size_t)r * g.N + n] = gemm_load(g, r, n);
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
  }
  return fn;
}

}  // namespace

int tma_encode_2d(CUtensorMap *m, const void *base, int is_fp16, unsigned long long rows, int cols, int box_rows,
                  int box_cols) {
  auto enc = get_encode();
  if (!enc) { g_last_cuda_error = 99999; return CORUN_ECUDA; }
  if (((uintptr_t)base & 15u) || (cols % 8) || (box_cols * 2 != 128 && box_cols * 2 != 32) || box_rows > 256 || box_rows < 1)
    return CORUN_EINVAL;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, is_fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                   const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   box_cols * 2 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_32B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) g_last_cuda_error = 100000 + (int)r;
  return r == CUDA_SUCCESS ? CORUN_OK : CORUN_ECUDA;
}

int tma_encode_fp16_nd(CUtensorMap *m, const void *base, int nd, const unsigned long long *dims, const unsigned long long *strides,
                       const unsigned *box) {
  auto enc = get_encode();
  if (!enc) { g_last_cuda_error = 99999; return CORUN_ECUDA; }
  if (nd < 2 || nd > 5 || ((uintptr_t)base & 15u) || box[0] * 2 != 128) return CORUN_EINVAL;
  cuuint64_t d[5], s[4];
  cuuint32_t b[5], estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < nd; ++i) {
    if (dims[i] < 1 || box[i] < 1 || box[i] > 256) return CORUN_EINVAL;
    d[i] = dims[i];
    b[i] = box[i];
  }
  for (int i = 0; i < nd - 1; ++i) {
    if (strides[i] % 16) return CORUN_EINVAL;
    s[i] = strides[i];
  }
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, (cuuint32_t)nd, const_cast<void *>(base), d, s, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) g_last_cuda_error = 100000 + (int)r;
  return r == CUDA_SUCCESS ? CORUN_OK : CORUN_ECUDA;
}

int tma_encode_fp16_4d(CUtensorMap *m, const void *base, const unsigned long long dims[4], const unsigned long long strides[3],
                       const unsigned box[4]) {
  return tma_encode_fp16_nd(m, base, 4, dims, strides, box);
}

int gemm_encode_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows) {
  if (K % GEMM_BLOCK_K) return CORUN_EINVAL;
  return tma_encode_2d(m, base, 0, (unsigned long long)rows, K, box_rows, GEMM_BLOCK_K);
}

// Activation rows per TMA box and activation bytes per stage: up to 64 padded rows one stacked tile (hi rows 0..,
// lo rows 64..), 65..128 rows two stacked tiles of 64 rows each (a box of 64 rows per half; the last box reaches
// past the matrix when BN < 128: those rows arrive as zeros), above that a hi and a lo box of 128 rows per row block.
static int gemm_x_box_rows(int BN) { return BN <= 64 ? BN : BN <= 128 ? 64 : GEMM_ROW_BLOCK; }
static size_t gemm_x_stage_bytes(int BN) {
  return BN <= 64 ? (size_t)A_BLOCK_BYTES : BN <= 128 ? 2 * (size_t)A_BLOCK_BYTES : 4 * (size_t)A_BLOCK_BYTES;
}

int gemm_plan_fill(GemmPlan *p, const void *W, int N, int K, const void *Xhi, const void *Xlo, int R, int BN,
                   float *direct, float *ws, int num_sms, int *tab, int tab_cap, int *tab_ints) {
  if (N <= 0 || K <= 0 || K % GEMM_BLOCK_K || BN % 16 || BN < 16 || BN > 256 || R < 1 || R > BN) return CORUN_EINVAL;
  p->N = N; p->K = K; p->R = R; p->BN = BN;
  p->n_tiles = (N + GEMM_TILE_N - 1) / GEMM_TILE_N;
  p->KB = K / GEMM_BLOCK_K;
  const long long total = (long long)p->n_tiles * p->KB;
  p->grid = (int)(total < num_sms ? total : num_sms);
  // With several CTAs per tile the ranges are cut tile by tile (the same number of CTAs for every tile, a few
  // SMs left out): no CTA then crosses a tile boundary, so none has two epilogues in a row, and above 128
  // rows -- where the two row blocks of a tile fill TMEM and the epilogue of a segment cannot overlap the MMAs
  // of the next -- none stops in the middle of its range.
  const int per_tile = p->grid >= 2 * p->n_tiles ? p->grid / p->n_tiles : 0;
  if (per_tile) p->grid = per_tile * p->n_tiles;
  if (total * (long long)p->grid >= (1ll << 31)) return CORUN_EINVAL;
  const size_t stage = (size_t)W_TILE_BYTES + gemm_x_stage_bytes(BN);
  // the MMA always reads 128 activation rows: leave that much readable behind the last stage
  int stages = (int)((GEMM_MAX_DYN_SMEM - 1024 - A_BLOCK_BYTES) / stage);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return CORUN_EINVAL;
  p->stages = stages;
  p->smem_bytes = stage * stages + A_BLOCK_BYTES + 1024;
  p->tmem_cols = 512;   // two accumulator buffers (<= 128 rows) or two row blocks
  // kind::f16 instruction descriptor: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1),
  // both K-major (bits 15, 16 = 0), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
  p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GEMM_TILE_N >> 3) << 17) |
             ((uint32_t)(GEMM_ROW_BLOCK >> 4) << 24);
  p->direct = direct;
  p->ws = ws;
  int rc;
  if ((rc = gemm_encode_map(&p->tmW, W, N, K, GEMM_TILE_N)) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmHi, Xhi, BN, K, gemm_x_box_rows(BN))) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmLo, Xlo, BN, K, gemm_x_box_rows(BN))) != 0) return rc;

  const int n_ints = p->grid + 1 + 3 * p->n_tiles;
  if (n_ints > tab_cap) return CORUN_ELIMIT;
  int *cs = tab, *cb = cs + p->grid + 1, *ce = cb + p->n_tiles, *sp = ce + p->n_tiles;
  for (int c = 0; c <= p->grid; ++c)
    cs[c] = per_tile ? (c / per_tile) * p->KB + (int)((long long)(c % per_tile) * p->KB / per_tile)
                     : (int)((long long)c * total / p->grid);
  p->n_split_tiles = 0;
  for (int t = 0, c = 0; t < p->n_tiles; ++t) {
    const int first = t * p->KB, last = first + p->KB - 1;
    while (cs[c + 1] <= first) ++c;
    cb[t] = 2 * c + (cs[c] < first ? 1 : 0);   // a CTA that began before the tile wrote its second slot
    int d = c;
    while (cs[d + 1] <= last) ++d;
    ce[t] = d;
    if (c != d) sp[p->n_split_tiles++] = t;
  }
  *tab_ints = n_ints;
  return CORUN_OK;
}

void gemm_plan_bind_tables(GemmPlan *p, int *d_tab) {
  p->d_cta_start = d_tab;
  p->d_tile_first = d_tab + p->grid + 1;
  p->d_tile_cend = p->d_tile_first + p->n_tiles;
  p->d_split_tiles = p->d_tile_cend + p->n_tiles;
}

int gemm_plan_create(GemmPlan *p, const void *W, int N, int K, const void *Xhi, const void *Xlo, int R, int BN,
                     float *direct, float *ws, int num_sms) {
  if (N <= 0 || K <= 0 || K % GEMM_BLOCK_K) return CORUN_EINVAL;
  const int n_tiles = (N + GEMM_TILE_N - 1) / GEMM_TILE_N;
  std::vector<int> tab((size_t)num_sms + 1 + 3 * (size_t)n_tiles);
  int n_ints = 0;
  int rc = gemm_plan_fill(p, W, N, K, Xhi, Xlo, R, BN, direct, ws, num_sms, tab.data(), (int)tab.size(), &n_ints);
  if (rc != CORUN_OK) return rc;
  int *d_tab = nullptr;
  if (cudaMalloc(&d_tab, (size_t)n_ints * sizeof(int)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t me = cudaMemcpy(d_tab, tab.data(), (size_t)n_ints * sizeof(int), cudaMemcpyHostToDevice);
  if (me != cudaSuccess) { g_last_cuda_error = (int)me; cudaFree(d_tab); return CORUN_ECUDA; }
  gemm_plan_bind_tables(p, d_tab);
  cudaError_t ae = gemm_prepare_kernel();
  if (ae != cudaSuccess) { g_last_cuda_error = (int)ae; return CORUN_ECUDA; }
  return CORUN_OK;
}

int gemm_swiglu_half(int F, int num_sms) {
  int half = ((F + num_sms - 1) / num_sms + 7) / 8 * 8;
  if (half < 64) half = 64;
  if (half > GEMM_TILE_N / 2) half = GEMM_TILE_N / 2;
  return half;
}

int gemm_plan_create_swiglu(GemmPlan *p, const void *W, int F, int K, const void *Xhi, const void *Xlo, int R, int BN,
                            __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int num_sms) {
  if (F <= 0 || F % 8 || K <= 0 || K % GEMM_BLOCK_K || BN % 16 || BN < 16 || BN > 256 || R < 1 || R > BN || !out_hi || !out_lo ||
      num_sms < 1)
    return CORUN_EINVAL;
  // as many whole tiles as there are SMs, if the matrix is large enough: the narrowest tile (a multiple of 8 gate
  // rows, at least 64) that still gives every CTA at most one
  const int HALF = gemm_swiglu_half(F, num_sms);
  p->sw_half = HALF;
  p->N = 2 * F; p->K = K; p->R = R; p->BN = BN;
  p->n_tiles = (F + HALF - 1) / HALF;
  p->KB = K / GEMM_BLOCK_K;
  p->grid = p->n_tiles < num_sms ? p->n_tiles : num_sms;
  if ((long long)p->n_tiles * p->KB >= (1ll << 31)) return CORUN_EINVAL;
  const size_t stage = (size_t)2 * HALF * GEMM_BLOCK_K * 2 + gemm_x_stage_bytes(BN);
  int stages = (int)((GEMM_MAX_DYN_SMEM - 1024 - A_BLOCK_BYTES) / stage);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return CORUN_EINVAL;
  p->stages = stages;
  p->smem_bytes = stage * stages + A_BLOCK_BYTES + 1024;
  p->tmem_cols = 512;
  p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * HALF) >> 3) << 17) |
             ((uint32_t)(GEMM_ROW_BLOCK >> 4) << 24);
  p->direct = nullptr;
  p->ws = nullptr;
  p->sw_hi = out_hi;
  p->sw_lo = out_lo;
  int rc;
  if ((rc = gemm_encode_map(&p->tmW, W, 2 * F, K, HALF)) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmHi, Xhi, BN, K, gemm_x_box_rows(BN))) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmLo, Xlo, BN, K, gemm_x_box_rows(BN))) != 0) return rc;
  // whole tiles only: CTA c takes tiles [c * n_tiles / grid, (c + 1) * n_tiles / grid)
  std::vector<int> tab((size_t)p->grid + 1);
  for (int c = 0; c <= p->grid; ++c) tab[(size_t)c] = (int)((long long)c * p->n_tiles / p->grid) * p->KB;
  int *d_tab = nullptr;
  if (cudaMalloc(&d_tab, tab.size() * sizeof(int)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t me = cudaMemcpy(d_tab, tab.data(), tab.size() * sizeof(int), cudaMemcpyHostToDevice);
  if (me != cudaSuccess) { g_last_cuda_error = (int)me; cudaFree(d_tab); return CORUN_ECUDA; }
  p->d_cta_start = d_tab;
  p->d_tile_first = p->d_tile_cend = p->d_split_tiles = nullptr;
  p->n_split_tiles = 0;
  cudaError_t ae = gemm_prepare_kernel();
  if (ae != cudaSuccess) { g_last_cuda_error = (int)ae; return CORUN_ECUDA; }
  return CORUN_OK;
}

int gemm_swiglu_blocks_half(int Fb, int n_blocks, int num_sms) {
  // the widest tile (a multiple of 8 gate rows that divides Fb, 64..128) for which the busiest CTA streams the
  // fewest weight rows; wider tiles mean fewer MMA instructions per byte, so ties go to the wider one
  int best = 0;
  long long best_cost = 0;
  for (int half = GEMM_TILE_N / 2; half >= 64; half -= 8) {
    if (Fb % half) continue;
    const long long tiles = (long long)n_blocks * (Fb / half);
    const long long cost = (tiles + num_sms - 1) / num_sms * half;
    if (!best || cost < best_cost) { best = half; best_cost = cost; }
  }
  return best;
}

int gemm_plan_create_swiglu_blocks(GemmPlan *p, const void *W, int n_blocks, int Fb, int K, const void *Xhi, const void *Xlo,
                                   int R, int BN, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, const float *row_scale,
                                   int num_sms) {
  if (n_blocks < 1 || Fb <= 0 || Fb % 8 || K <= 0 || K % GEMM_BLOCK_K || BN % 16 || BN < 16 || BN > 256 || R < 1 || R > BN ||
      !out_hi || !out_lo || !row_scale || num_sms < 1)
    return CORUN_EINVAL;
  const int HALF = gemm_swiglu_blocks_half(Fb, n_blocks, num_sms);
  if (!HALF) return CORUN_EINVAL;
  p->sw_half = HALF;
  p->N = n_blocks * 2 * Fb; p->K = K; p->R = R; p->BN = BN;
  p->n_tiles = n_blocks * (Fb / HALF);
  p->KB = K / GEMM_BLOCK_K;
  p->grid = p->n_tiles < num_sms ? p->n_tiles : num_sms;
  if ((long long)p->n_tiles * p->KB >= (1ll << 31)) return CORUN_EINVAL;
  const size_t stage = (size_t)2 * HALF * GEMM_BLOCK_K * 2 + gemm_x_stage_bytes(BN);
  int stages = (int)((GEMM_MAX_DYN_SMEM - 1024 - A_BLOCK_BYTES) / stage);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return CORUN_EINVAL;
  p->stages = stages;
  p->smem_bytes = stage * stages + A_BLOCK_BYTES + 1024;
  p->tmem_cols = 512;
  p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * HALF) >> 3) << 17) |
             ((uint32_t)(GEMM_ROW_BLOCK >> 4) << 24);
  p->direct = nullptr;
  p->ws = nullptr;
  p->sw_hi = out_hi;
  p->sw_lo = out_lo;
  p->row_keep = row_scale;
  p->keep_pitch = n_blocks;
  p->keep_div = Fb / HALF;
  int rc;
  if ((rc = gemm_encode_map(&p->tmW, W, n_blocks * 2 * Fb, K, HALF)) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmHi, Xhi, BN, K, gemm_x_box_rows(BN))) != 0) return rc;
  if ((rc = gemm_encode_map(&p->tmLo, Xlo, BN, K, gemm_x_box_rows(BN))) != 0) return rc;
  // whole tiles only: CTA c takes tiles [c * n_tiles / grid, (c + 1) * n_tiles / grid)
  std::vector<int> tab((size_t)p->grid + 1);
  for (int c = 0; c <= p->grid; ++c) tab[(size_t)c] = (int)((long long)c * p->n_tiles / p->grid) * p->KB;
  int *d_tab = nullptr;
  if (cudaMalloc(&d_tab, tab.size() * sizeof(int)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t me = cudaMemcpy(d_tab, tab.data(), tab.size() * sizeof(int), cudaMemcpyHostToDevice);
  if (me != cudaSuccess) { g_last_cuda_error = (int)me; cudaFree(d_tab); return CORUN_ECUDA; }
  p->d_cta_start = d_tab;
  p->d_tile_first = p->d_tile_cend = p->d_split_tiles = nullptr;
  p->n_split_tiles = 0;
  cudaError_t ae = gemm_prepare_kernel();
  if (ae != cudaSuccess) { g_last_cuda_error = (int)ae; return CORUN_ECUDA; }
  return CORUN_OK;
}

int gemm_plan_create_grouped(GemmPlan *p, const void *W, long long w_rows, int w_cols, int N, int K, const void *Xhi,
                             const void *Xlo, int n_groups, int BN, float *direct, const int *group_tab, int num_sms) {
  if (N <= 0 || N % GEMM_TILE_N || K <= 0 || K % GEMM_BLOCK_K || w_cols % GEMM_BLOCK_K || BN % 16 || BN < 16 || BN > 64 ||
      n_groups < 1 || !group_tab || w_rows < N || num_sms < 1)
    return CORUN_EINVAL;
  p->N = N; p->K = K; p->R = BN; p->BN = BN;
  p->n_tiles = n_groups * (N / GEMM_TILE_N);
  p->KB = K / GEMM_BLOCK_K;
  p->grid = p->n_tiles < num_sms ? p->n_tiles : num_sms;
  p->keep_pitch = n_groups;                         // where the table's count of groups in use sits
  const size_t stage = (size_t)GEMM_TILE_N * GEMM_BLOCK_K * 2 + (size_t)GEMM_ROW_BLOCK * GEMM_BLOCK_K * 2;
  int stages = (int)((GEMM_MAX_DYN_SMEM - 1024 - A_BLOCK_BYTES) / stage);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  p->stages = stages;
  p->smem_bytes = stage * stages + A_BLOCK_BYTES + 1024;
  p->tmem_cols = 512;
  p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GEMM_TILE_N >> 3) << 17) |
             ((uint32_t)(GEMM_ROW_BLOCK >> 4) << 24);
  p->direct = direct;
  p->ws = nullptr;
  p->group_tab = group_tab;
  p->tiles_per_group = N / GEMM_TILE_N;
  int rc;
  if ((rc = tma_encode_2d(&p->tmW, W, 0, (unsigned long long)w_rows, w_cols, GEMM_TILE_N, GEMM_BLOCK_K)) != 0) return rc;
  if ((rc = tma_encode_2d(&p->tmHi, Xhi, 0, (unsigned long long)n_groups * BN, K, BN, GEMM_BLOCK_K)) != 0) return rc;
  if ((rc = tma_encode_2d(&p->tmLo, Xlo, 0, (unsigned long long)n_groups * BN, K, BN, GEMM_BLOCK_K)) != 0) return rc;
  // every CTA's range is exactly one tile
  std::vector<int> tab((size_t)p->grid + 1);
  for (int c = 0; c <= p->grid; ++c) tab[(size_t)c] = c * p->KB;
  int *d_tab = nullptr;
  if (cudaMalloc(&d_tab, tab.size() * sizeof(int)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t me = cudaMemcpy(d_tab, tab.data(), tab.size() * sizeof(int), cudaMemcpyHostToDevice);
  if (me != cudaSuccess) { g_last_cuda_error = (int)me; cudaFree(d_tab); return CORUN_ECUDA; }
  p->d_cta_start = d_tab;
  p->d_tile_first = p->d_tile_cend = p->d_split_tiles = nullptr;
  p->n_split_tiles = 0;
  cudaError_t ae = gemm_prepare_kernel();
  if (ae != cudaSuccess) { g_last_cuda_error = (int)ae; return CORUN_ECUDA; }
  return CORUN_OK;
}

int gemm_plan_create_grouped_swiglu(GemmPlan *p, const void *W, long long w_rows, int F, int K, int half, const void *Xhi,
                                    const void *Xlo, int n_groups, int BN, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                    const float *row_scale, const int *group_tab, int num_sms) {
  if (F <= 0 || half < 64 || half > GEMM_TILE_N / 2 || half % 8 || F % half || K <= 0 || K % GEMM_BLOCK_K || BN % 16 || BN < 16 ||
      BN > 64 || n_groups < 1 || !group_tab || !out_hi || !out_lo || !row_scale || w_rows < 2 * F || num_sms < 1)
    return CORUN_EINVAL;
  p->sw_half = half;
  p->N = 2 * F; p->K = K; p->R = BN; p->BN = BN;
  p->tiles_per_group = F / half;
  p->n_tiles = n_groups * p->tiles_per_group;
  p->KB = K / GEMM_BLOCK_K;
  p->grid = p->n_tiles < num_sms ? p->n_tiles : num_sms;
  p->keep_pitch = n_groups;
  const size_t stage = (size_t)2 * half * GEMM_BLOCK_K * 2 + (size_t)A_BLOCK_BYTES;
  int stages = (int)((GEMM_MAX_DYN_SMEM - 1024 - A_BLOCK_BYTES) / stage);
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  p->stages = stages;
  p->smem_bytes = stage * stages + A_BLOCK_BYTES + 1024;
  p->tmem_cols = 512;
  p->idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * half) >> 3) << 17) | ((uint32_t)(GEMM_ROW_BLOCK >> 4) << 24);
  p->direct = nullptr;
  p->ws = nullptr;
  p->sw_hi = out_hi;
  p->sw_lo = out_lo;
  p->row_keep = row_scale;
  p->group_tab = group_tab;
  int rc;
  if ((rc = tma_encode_2d(&p->tmW, W, 0, (unsigned long long)w_rows, K, half, GEMM_BLOCK_K)) != 0) return rc;
  if ((rc = tma_encode_2d(&p->tmHi, Xhi, 0, (unsigned long long)n_groups * BN, K, BN, GEMM_BLOCK_K)) != 0) return rc;
  if ((rc = tma_encode_2d(&p->tmLo, Xlo, 0, (unsigned long long)n_groups * BN, K, BN, GEMM_BLOCK_K)) != 0) return rc;
  p->d_cta_start = p->d_tile_first = p->d_tile_cend = p->d_split_tiles = nullptr;   // the kernel derives its tiles itself
  p->n_split_tiles = 0;
  cudaError_t ae = gemm_prepare_kernel();
  if (ae != cudaSuccess) { g_last_cuda_error = (int)ae; return CORUN_ECUDA; }
  return CORUN_OK;
}

cudaError_t gemm_prepare_kernel() {
  cudaError_t e = cudaFuncSetAttribute(gemm_streamk_kernel<false, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, false, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, true, false, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<false, true, false, true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_streamk_kernel<true, true, false, true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_MAX_DYN_SMEM);
  return e;
}

void gemm_plan_destroy(GemmPlan *p) {
  if (p->d_cta_start) cudaFree(p->d_cta_start);
  p->d_cta_start = nullptr;
}

cudaError_t gemm_launch(const GemmPlan &p, const CUtensorMap *tmW_override, int *d_status, cudaStream_t st,
                        unsigned long long *trace, bool pdl) {
  const bool masked = p.row_keep != nullptr, stacked = p.BN <= 64;
  auto go = [&](auto kernel) {
    return launch_k(kernel, dim3(p.grid), dim3(GEMM_THREADS), p.smem_bytes, st, pdl, tmW_override ? *tmW_override : p.tmW,
                    p.tmHi, p.tmLo, p.direct, p.ws, p.d_cta_start, p.N, p.KB, p.BN, p.R, p.stages, p.tmem_cols, p.idesc,
                    p.row_keep, p.keep_pitch, p.keep_div, p.group_tab, p.tiles_per_group, d_status, trace, p.sw_hi, p.sw_lo,
                    p.sw_half, p.row_blocks);
  };
  if (!p.group_tab && p.BN > 64 && p.BN <= 128) {   // two stacked blocks of 64 rows
    if (p.sw_hi) return masked ? go(gemm_streamk_kernel<true, true, false, true, 2>) : go(gemm_streamk_kernel<false, true, false, true, 2>);
    return masked ? go(gemm_streamk_kernel<true, true, false, false, 2>) : go(gemm_streamk_kernel<false, true, false, false, 2>);
  }
  if (p.group_tab && p.sw_hi) return go(gemm_streamk_kernel<false, true, true, true>);
  if (p.sw_hi && masked) return stacked ? go(gemm_streamk_kernel<true, true, false, true>) : go(gemm_streamk_kernel<true, false, false, true>);
  if (p.sw_hi) return stacked ? go(gemm_streamk_kernel<false, true, false, true>) : go(gemm_streamk_kernel<false, false, false, true>);
  if (p.group_tab) return go(gemm_streamk_kernel<false, true, true, false>);
  if (masked) return stacked ? go(gemm_streamk_kernel<true, true, false, false>) : go(gemm_streamk_kernel<true, false, false, false>);
  return stacked ? go(gemm_streamk_kernel<false, true, false, false>) : go(gemm_streamk_kernel<false, false, false, false>);
}

cudaError_t gemm_fixup_launch(const GemmPlan &p, cudaStream_t st, bool pdl) {
  if (p.n_split_tiles == 0) return cudaSuccess;
  return launch_k(gemm_fixup_kernel, dim3(p.n_split_tiles, p.R), dim3(GEMM_TILE_N), 0, st, pdl, p.out(), p.direct,
                  p.d_split_tiles);
}

}  // namespace corun
