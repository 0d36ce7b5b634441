// Multi-head latent attention (MLA) for one query token per row at decode time, absorbed form, over a PAGED
// latent cache, on tcgen05 / TMEM / TMA (sm_100a).
//
// Per cached token the cache holds the latent c_t [d_c] followed by the shared rotary key r_t [d_r] (fp16); all
// heads of a row share it.  With the up-projections absorbed into the query, a head's scores and output are
//     s_{h,t} = (q_lat[h] . c_t + q_rope[h] . r_t) * scale,   p_h = softmax_t(s_h),   o_lat[h] = sum_t p_{h,t} c_t.
//
// An item is (row, split of 256 cached tokens = 16 pages); the items of a call are listed row by row and every
// CTA (one per SM) takes one contiguous stretch of the list.  What bounds this op on the tensor cores is the
// NUMBER of MMA instructions (each takes ~150 cycles whatever its shape), so the products are arranged to need
// few: the 16 heads (as fp16 hi + lo rows, 32 rows of a 64-row operand) are the M side, the tokens and the
// latent dims the wide N side:
//   scores   S[32 x 256 tokens] = Q[32 x 576] * [C | R]^T    4 MMAs (K = 16 each) per block of 64 dims: 36
//   output   O[32 x 512 dims]  = P[32 x 256 tokens] * C      per half of 256 dims one MMA per page: 32
// The latent is streamed TWICE through a ring of four 32 KiB slots: once for the scores as K-major blocks of
// [256 tokens x 64 dims] (one [16 x 64] box per page), and once more -- from L2 by then -- for the output as
// units of four pages x 256 dims, each page fetched by ONE 4-dimensional box [2 groups][4 blocks][8 tokens][64 dims]
// that lands as the MN-major N operand of its MMA.  The output product of an item is issued after the scores of
// the NEXT item, so the tensor pipe works on one while the softmax of the other runs.
//   warp 0             producer: block-table lookups and TMA loads;
//   warp 1             issues the MMAs;
//   warps 2, 3, 6, 7   build the query tile (fp16 hi / lo rows, 128-byte swizzle) when the row changes;
//   warps 4, 5, 8, 9   softmax: a 64-row accumulator keeps rows 0-15 / 16-31 in lanes 0-15 of TMEM lane quarters
//                      0 / 1; row 2h is head h's hi part, row 2h + 1 its lo part.  Warps 4, 5 take tokens 0-127,
//                      warps 8, 9 tokens 128-255: exact maximum, weights as an fp16 hi / lo operand tile, sum;
//   warps 12, 13, 16, 17  read the output accumulator, add the hi and lo rows and store the split's partial.
// A second kernel, one warp per (row, head), combines a row's splits in ascending order.
//
// Invariance: the split size is fixed, the split count is a function of the row's own context length, every
// reduction inside an item has one fixed order and the combine is ascending; which CTA computes an item has no
// influence on any value.  Every wait is bounded.
#include <cuda_fp16.h>
#include <math_constants.h>

#include "../../include/corun.h"
#include "../../include/corun_mla.h"
#include "gemm.cuh"
#include "launch.cuh"
#include "mla.cuh"
#include "ptx.cuh"

namespace corun {
namespace {

constexpr int MP_T = 256;                    // tokens per item
constexpr int MP_PAGE = 16;                  // tokens per page
constexpr int MP_PAGES = MP_T / MP_PAGE;
constexpr int MP_BOX = MP_PAGE * 128;        // bytes of one [16 tokens x 64 dims] box
constexpr int MP_SLOT = MP_T * 128;          // bytes of a ring slot: [256 tokens x 64 dims] or 4 pages x 256 dims
constexpr int MP_RING = 4;
constexpr int MP_QBLK = 32 * 128;            // bytes of one [32 rows x 64 dims] block of the query / weight tiles
constexpr int MP_PBUF = (MP_T / 64 + 1) * MP_QBLK;   // one weight tile: 4 blocks of 64 tokens + overrun
constexpr int MP_MAXH = 16;                  // heads (hi + lo rows: 32 of the operand's 64)
constexpr int MP_MAXB = 1024;                // rows per call
constexpr int MP_ITEM_COST = 512;            // what an item costs beyond its tokens, in tokens (score MMAs, waits and hand-offs do not shrink with it)
constexpr int MP_THREADS = 576;
constexpr uint32_t MP_TMEM_COLS = 512;       // S: 256 columns, O: 256 columns
// shared memory: [ring][query tile: 9 blocks + overrun][two weight tiles]
constexpr int MP_OFF_Q = MP_RING * MP_SLOT;
constexpr int MP_OFF_P = MP_OFF_Q + 10 * MP_QBLK;
constexpr int MP_SMEM = MP_OFF_P + 2 * MP_PBUF + 1024;

__device__ __forceinline__ uint32_t mp_swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }
__device__ __forceinline__ float mp_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// two fp32 -> packed fp16 hi parts and packed fp16 lo parts (x = hi + lo up to 2^-22 |x|)
__device__ __forceinline__ void mp_split2(float x0, float x1, uint32_t &hi, uint32_t &lo) {
  const __half2 h = __floats2half2_rn(x0, x1);
  const float2 f = __half22float2(h);
  const __half2 l = __floats2half2_rn(x0 - f.x, x1 - f.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}
// 32 lanes x 32 consecutive 32-bit columns
__device__ __forceinline__ void mp_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  tmem_ld16(taddr, *reinterpret_cast<uint32_t(*)[16]>(&r[0]));
  tmem_ld16(taddr + 16, *reinterpret_cast<uint32_t(*)[16]>(&r[16]));
}

// part_ml [B][max_splits][n_heads] (max in the base-2 domain, sum), part_o [B][max_splits][n_heads][d_c]
__global__ void __launch_bounds__(MP_THREADS, 1)
mla_paged_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmV, const float *__restrict__ q_lat,
                 long long q_rs, long long q_hs, const float *__restrict__ q_rope, const int *__restrict__ block_table, int max_blocks,
                 const int *__restrict__ ctx, const int *__restrict__ row_slot, const int *__restrict__ row_pos,
                 const int *__restrict__ row_active, int B, int n_heads, int d_c, int d_r, float scale_log2e, int max_splits,
                 float2 *__restrict__ part_ml, float *__restrict__ part_o, int *status, int page_run) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MP_RING], empty_bar[MP_RING];
  __shared__ __align__(8) uint64_t q_ready_bar, q_free_bar, s_full_bar, s_free_bar, p_ready_bar, o_full_bar, o_free_bar, x_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ float xs_mx[2][32], xs_sum[2][32];   // the two token halves of an item exchange maximum and sum
  __shared__ int row_start[MP_MAXB + 1];           // first item of every row
  __shared__ int row_ctx[MP_MAXB];                 // cached tokens of every row (cut to the block table's reach)
  __shared__ int cost_start[MP_MAXB + 1];          // cost of all items before the row (tokens + MP_ITEM_COST per item)
  __shared__ int my_items[2];                      // this CTA's stretch of the item list
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < MP_RING; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    mbar_init(smem_u32(&q_ready_bar), 4);
    mbar_init(smem_u32(&q_free_bar), 1);
    mbar_init(smem_u32(&s_full_bar), 1);
    mbar_init(smem_u32(&s_free_bar), 4);
    mbar_init(smem_u32(&p_ready_bar), 4);
    mbar_init(smem_u32(&o_full_bar), 1);
    mbar_init(smem_u32(&o_free_bar), 4);
    mbar_init(smem_u32(&x_bar), 4);
    fence_mbar_init();
    fence_proxy_async();
    prefetch_tensormap(&tmC);
    prefetch_tensormap(&tmV);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_base_s), MP_TMEM_COLS);
    tmem_relinquish();
  } else if (warp >= 4) {
    // the operand tiles start out as zeros: rows of absent heads and rope columns beyond d_r stay zero
    uint4 *z = reinterpret_cast<uint4 *>(base_ptr + MP_OFF_Q);
    for (int i = tid - 128; i < (10 * MP_QBLK + 2 * MP_PBUF) / 16; i += MP_THREADS - 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // (programmatic launch) everything above reads nothing that another kernel writes: it runs while the kernels before
  // this one drain.  The inputs are taken through after_wait so that no load is moved up across the wait.
  griddep_wait();
  q_lat = after_wait(q_lat); q_rope = after_wait(q_rope); block_table = after_wait(block_table); ctx = after_wait(ctx);
  row_slot = after_wait(row_slot); row_pos = after_wait(row_pos); row_active = after_wait(row_active);
  if (warp == 2) {
    // items per row -> first item of every row (one warp, rows in chunks of 32, ascending)
    int run = 0, crun = 0;
    for (int r0 = 0; r0 < B; r0 += 32) {
      const int r = r0 + lane;
      int n = 0, cst = 0;
      if (r < B) {
        int c = row_pos ? (row_active[r] ? row_pos[r] + 1 : 0) : ctx[r];
        c = c < 0 ? 0 : (c > max_blocks * MP_PAGE ? max_blocks * MP_PAGE : c);
        n = (c + MP_T - 1) / MP_T;
        if (n > max_splits) { n = max_splits; c = n * MP_T; }
        row_ctx[r] = c;
        cst = c + n * MP_ITEM_COST;
      }
      int inc = n, cinc = cst;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, inc, o), cv = __shfl_up_sync(0xffffffffu, cinc, o);
        if (lane >= o) { inc += v; cinc += cv; }
      }
      if (r < B) { row_start[r] = run + inc - n; cost_start[r] = crun + cinc - cst; }
      run += __shfl_sync(0xffffffffu, inc, 31);
      crun += __shfl_sync(0xffffffffu, cinc, 31);
    }
    __syncwarp();
    if (lane == 0) {
      row_start[B] = run;
      cost_start[B] = crun;
      // The CTAs' stretches are cut where the items' accumulated cost passes k / grid of the total (an item goes to
      // the CTA in whose share it starts), so that CTAs with cheaper (shorter) items take more of them.  Which CTA
      // computes an item has no influence on any value.
      auto bound = [&](int k) {
        if (k >= (int)gridDim.x) return run;
        const long long t = ((long long)crun * k + gridDim.x - 1) / gridDim.x;
        int lo = 0, hi = B;                          // last row whose cost_start is <= t
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (cost_start[mid] <= t) lo = mid; else hi = mid;
        }
        const int n_r = row_start[lo + 1] - row_start[lo];
        const int sidx = (int)((t - cost_start[lo] + (MP_T + MP_ITEM_COST) - 1) / (MP_T + MP_ITEM_COST));
        return sidx >= n_r ? row_start[lo + 1] : row_start[lo] + sidx;
      };
      my_items[0] = bound((int)blockIdx.x);
      my_items[1] = bound((int)blockIdx.x + 1);
    }
  }
  __syncthreads();
  const uint32_t tmem_base = tmem_base_s;
  const uint32_t s_tmem = tmem_base, o_tmem = tmem_base + 256;
  const int n_items = row_start[B];
  const int item_lo = my_items[0], item_hi = n_items > 0 ? my_items[1] : 0;
  const int NLB = d_c / 64;                    // latent blocks (1, 2, 4 or 8)
  const int n_half = d_c > 256 ? 2 : 1, BPH = NLB / n_half, NH = d_c / n_half;   // output halves, blocks and dims per half
  bool failed = false;
  int cur_row = 0;
  auto locate = [&](int item, int &r, int &split) {   // items ascend: the row pointer only moves forward
    while (item >= row_start[cur_row + 1]) ++cur_row;
    r = cur_row;
    split = item - row_start[cur_row];
  };
  auto tokens_of = [&](int r, int split) { return min(MP_T, row_ctx[r] - split * MP_T); };

  if (warp == 0) {
    // ---------------- producer ----------------
    // the score pass leaves the blocks in L2 for the output pass, which is the last use
    const uint64_t pol_keep = l2_policy_evict_last(), pol_drop = l2_policy_evict_first();
    int u = 0, prev_page = 0, prev_np = 0;
    auto slot_free = [&](int unit) {
      if (unit < MP_RING) return true;
      bool ok = mbar_wait(smem_u32(&empty_bar[unit % MP_RING]), (uint32_t)(unit / MP_RING - 1) & 1u, &abort_flag);
      return (bool)__all_sync(0xffffffffu, ok);
    };
    auto pages_of = [&](int it, int &n) {             // lane l: page l of the item (0 beyond its pages)
      if (it >= item_hi) { n = 0; return 0; }
      int r, split;
      locate(it, r, split);
      n = (tokens_of(r, split) + MP_PAGE - 1) / MP_PAGE;
      const int tr = row_slot ? __ldg(row_slot + r) : r;     // whose block table the row reads
      return lane < n ? __ldg(block_table + (size_t)tr * max_blocks + split * MP_PAGES + lane) : 0;
    };
    int np_ahead = 0, page_ahead = pages_of(item_lo, np_ahead);
    for (int it = item_lo; it <= item_hi && !failed; ++it) {
      const int page = page_ahead, np = np_ahead;      // looked up one item ahead of its use
      page_ahead = pages_of(it + 1, np_ahead);
      if (it < item_hi) {
        // page_run consecutive pool pages per box (4: the table's pages come in aligned runs of four, so one box of
        // 64 tokens fetches what four boxes of 16 would: the TMA unit is bound by the number of boxes)
        const int nbx = (np + page_run - 1) / page_run;
        const int bpage = __shfl_sync(0xffffffffu, page, (page_run * lane) & 31);
        for (int j = 0; j <= NLB; ++j, ++u) {           // latent blocks, then the rope block
          if (!slot_free(u)) { failed = true; break; }
          const uint32_t bar = smem_u32(&full_bar[u % MP_RING]);
          if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)(nbx * page_run * MP_BOX));
          __syncwarp();
          if (lane < nbx) {
            const uint32_t dst = base + (uint32_t)(u % MP_RING) * MP_SLOT + (uint32_t)(lane * page_run) * MP_BOX;
            if (page_run == 4)   // block-major runs: rows of 64 dims, block j of run r = rows ((r * blocks + j) * 64 ..
              tma_load_2d(dst, &tmC, 0, ((bpage >> 2) * (NLB + 1) + j) * 64, bar, pol_keep);
            else
              tma_load_2d(dst, &tmC, j < NLB ? 64 * j : d_c, bpage * MP_PAGE, bar, pol_keep);
          }
        }
      }
      if (it > item_lo && !failed) {                     // the previous item's latent once more, page-major
        const int nu = (prev_np + 3) / 4;
        for (int hu = 0; hu < n_half * nu; ++hu, ++u) {
          const int half = hu / nu, uu = hu - half * nu;
          if (!slot_free(u)) { failed = true; break; }
          const int cnt = page_run == 4 ? 1 : min(4, prev_np - 4 * uu);   // boxes: a run of four pages is one
          const int pg = __shfl_sync(0xffffffffu, prev_page, (4 * uu + lane) & 31);
          const uint32_t bar = smem_u32(&full_bar[u % MP_RING]);
          if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)(cnt * page_run * BPH * MP_BOX));
          __syncwarp();
          if (lane < cnt) {
            const uint32_t dst = base + (uint32_t)(u % MP_RING) * MP_SLOT + (uint32_t)(lane * BPH) * MP_BOX;
            if (page_run == 4) tma_load_5d(dst, &tmV, 0, 0, half * BPH, 0, pg >> 2, bar, pol_drop);
            else tma_load_4d(dst, &tmV, 0, 0, half * BPH, pg * 2, bar, pol_drop);
          }
        }
      }
      prev_page = page;
      prev_np = np;
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      // D fp32, A and B fp16 (format 0), M = 64; scores: N = 256, both K-major; output: N = NH, B MN-major
      const uint32_t idesc_s = (1u << 4) | ((uint32_t)(MP_T >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);
      const uint32_t idesc_o = (1u << 4) | (1u << 16) | ((uint32_t)(NH >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);
      const uint32_t q_tile = base + MP_OFF_Q;
      int u = 0, n_q = 0, n_o = 0, last_row = -1, prev_np = 0;
      for (int it = item_lo; it <= item_hi && !failed; ++it) {
        int np = 0;
        if (it < item_hi) {
          int r, split;
          locate(it, r, split);
          np = (tokens_of(r, split) + MP_PAGE - 1) / MP_PAGE;
          if (r != last_row) {                       // the query tile of the new row
            if (!mbar_wait(smem_u32(&q_ready_bar), (uint32_t)n_q & 1u, &abort_flag)) { failed = true; break; }
            ++n_q;
            last_row = r;
          }
          if (it > item_lo && !mbar_wait(smem_u32(&s_free_bar), (uint32_t)(it - 1 - item_lo) & 1u, &abort_flag)) { failed = true; break; }
          tc_fence_after();
          for (int j = 0; j <= NLB; ++j, ++u) {      // query block NLB is the rope block
            const int slot = u % MP_RING;
            if (!mbar_wait(smem_u32(&full_bar[slot]), (uint32_t)(u / MP_RING) & 1u, &abort_flag)) { failed = true; break; }
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t a = umma_desc_sw128(q_tile + (uint32_t)j * MP_QBLK) + (uint64_t)(ks * 2);
              const uint64_t b = umma_desc_sw128(base + (uint32_t)slot * MP_SLOT) + (uint64_t)(ks * 2);
              umma_bf16(s_tmem, a, b, idesc_s, (j > 0 || ks > 0) ? 1u : 0u);
            }
            umma_commit(smem_u32(&empty_bar[slot]));
          }
          if (failed) break;
          umma_commit(smem_u32(&s_full_bar));
          if (it + 1 < item_hi && it + 1 >= row_start[r + 1]) umma_commit(smem_u32(&q_free_bar));   // the row's last scores
        }
        if (it > item_lo) {
          // ---- output of the previous item, half by half, once its weights are in their tile
          const int k = it - 1 - item_lo;
          if (!mbar_wait(smem_u32(&p_ready_bar), (uint32_t)k & 1u, &abort_flag)) { failed = true; break; }
          const uint32_t p_tile = base + MP_OFF_P + (uint32_t)(k & 1) * MP_PBUF;
          const int nu = (prev_np + 3) / 4;
          for (int half = 0; half < n_half && !failed; ++half, ++n_o) {
            if (n_o > 0 && !mbar_wait(smem_u32(&o_free_bar), (uint32_t)(n_o - 1) & 1u, &abort_flag)) { failed = true; break; }
            tc_fence_after();
            for (int uu = 0; uu < nu; ++uu, ++u) {
              const int slot = u % MP_RING;
              if (!mbar_wait(smem_u32(&full_bar[slot]), (uint32_t)(u / MP_RING) & 1u, &abort_flag)) { failed = true; break; }
              tc_fence_after();
              const int cnt = min(4, prev_np - 4 * uu);
              for (int pp = 0; pp < cnt; ++pp) {
                const int p = 4 * uu + pp;
                const uint64_t a = umma_desc_sw128(p_tile + (uint32_t)(p >> 2) * MP_QBLK) + (uint64_t)((p & 3) * 2);
                const uint64_t b = umma_desc_sw128_mn(base + (uint32_t)slot * MP_SLOT + (uint32_t)(pp * BPH) * MP_BOX, 1024u, (uint32_t)BPH * 1024u);
                umma_bf16(o_tmem, a, b, idesc_o, p > 0 ? 1u : 0u);
              }
              umma_commit(smem_u32(&empty_bar[slot]));
            }
            if (failed) break;
            umma_commit(smem_u32(&o_full_bar));
          }
        }
        prev_np = np;
      }
    }
  } else if (warp == 2 || warp == 3 || warp == 6 || warp == 7) {
    // ---------------- query tile ----------------
    // [block of 64 dims][row 2h = hi / 2h + 1 = lo][64 dims], 128-byte swizzle; chunks of 8 dims per thread
    const int qtid = ((warp & 1) + (warp >= 6 ? 2 : 0)) * 32 + lane;
    uint8_t *q_ptr = base_ptr + MP_OFF_Q;
    const int chunks = (d_c + d_r) >> 3, total = n_heads * chunks;
    int n_build = 0, last_row = -1;
    for (int it = item_lo; it < item_hi && !failed; ++it) {
      int r, split;
      locate(it, r, split);
      if (r == last_row) continue;
      if (n_build > 0) {                              // the previous row's last scores have read the tile
        bool ok = mbar_wait(smem_u32(&q_free_bar), (uint32_t)(n_build - 1) & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      for (int i0 = qtid; i0 < total; i0 += 3 * 128) {   // three chunks per thread at a time: their loads overlap
        float4 x0[3], x1[3];
        int hh[3], dd[3];
#pragma unroll
        for (int e = 0; e < 3; ++e) {
          const int i = i0 + e * 128;
          hh[e] = -1;
          if (i < total) {
            const int h = i / chunks, d = (i - h * chunks) << 3;
            const float *src = d < d_c ? q_lat + (size_t)r * q_rs + (size_t)h * q_hs + d : q_rope + ((size_t)r * n_heads + h) * d_r + (d - d_c);
            x0[e] = __ldg(reinterpret_cast<const float4 *>(src));
            x1[e] = __ldg(reinterpret_cast<const float4 *>(src) + 1);
            hh[e] = h;
            dd[e] = d;
          }
        }
#pragma unroll
        for (int e = 0; e < 3; ++e) {
          if (hh[e] < 0) continue;
          const int h = hh[e], d = dd[e];
          uint4 hi, lo;
          mp_split2(x0[e].x, x0[e].y, hi.x, lo.x);
          mp_split2(x0[e].z, x0[e].w, hi.y, lo.y);
          mp_split2(x1[e].x, x1[e].y, hi.z, lo.z);
          mp_split2(x1[e].z, x1[e].w, hi.w, lo.w);
          const int blk = d < d_c ? (d >> 6) : NLB, cc = d < d_c ? ((d & 63) >> 3) : ((d - d_c) >> 3);
          uint8_t *t = q_ptr + (size_t)blk * MP_QBLK;
          *reinterpret_cast<uint4 *>(t + mp_swz(2 * h, cc)) = hi;
          *reinterpret_cast<uint4 *>(t + mp_swz(2 * h + 1, cc)) = lo;
        }
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&q_ready_bar));
      ++n_build;
      last_row = r;
    }
  } else if (warp == 4 || warp == 5 || warp == 8 || warp == 9) {
    // ---------------- softmax ----------------
    const int q = warp & 3;                          // TMEM lane quarter: rows 16 q .. 16 q + 15 in lanes 0-15
    const int c = warp >= 8 ? 1 : 0;                 // token half of the item
    const int row16 = 16 * q + (lane & 15);          // operand / accumulator row of this lane
    const int head = row16 >> 1;                     // rows 2h (hi) and 2h + 1 (lo) belong to head h
    const bool head_ok = lane < 16 && head < n_heads;
    const bool even = (lane & 1) == 0;
    const uint32_t s_lane = s_tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(c * 128);
    for (int it = item_lo; it < item_hi && !failed; ++it) {
      const int k = it - item_lo;
      int r, split;
      locate(it, r, split);
      const int n_tok = tokens_of(r, split) - c * 128;   // valid tokens among this warp's 128
      {
        bool ok = mbar_wait(smem_u32(&s_full_bar), (uint32_t)k & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      tc_fence_after();
      float mx = -CUDART_INF_F;
      for (int c0 = 0; c0 < 128; c0 += 32) {         // pass 1: the exact maximum over the tokens
        uint32_t v[32];
        mp_tmem_ld32(s_lane + (uint32_t)c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float mine = __uint_as_float(v[j]);
          const float s = mine + __shfl_xor_sync(0xffffffffu, mine, 1);   // hi row + lo row
          if (c0 + j < n_tok) mx = fmaxf(mx, s);
        }
      }
      if (lane < 16) xs_mx[c][row16] = mx;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&x_bar));
      {
        bool ok = mbar_wait(smem_u32(&x_bar), (uint32_t)(2 * k) & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      mx = fmaxf(xs_mx[0][row16], xs_mx[1][row16]) * scale_log2e;   // scale > 0: the maximum commutes with it
      float sum = 0.f;
      uint8_t *p_row = base_ptr + MP_OFF_P + (size_t)(k & 1) * MP_PBUF + (size_t)(2 * c) * MP_QBLK;
      for (int c0 = 0; c0 < 128; c0 += 32) {         // pass 2: weights and their sum, tokens ascending
        uint32_t v[32];
        mp_tmem_ld32(s_lane + (uint32_t)c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int j8 = 0; j8 < 32; j8 += 8) {
          float p[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float mine = __uint_as_float(v[j8 + j]);
            const float s = mine + __shfl_xor_sync(0xffffffffu, mine, 1);
            p[j] = c0 + j8 + j < n_tok ? mp_ex2(fmaf(s, scale_log2e, -mx)) : 0.f;
            sum += p[j];
          }
          uint4 hi, lo;
          mp_split2(p[0], p[1], hi.x, lo.x);
          mp_split2(p[2], p[3], hi.y, lo.y);
          mp_split2(p[4], p[5], hi.z, lo.z);
          mp_split2(p[6], p[7], hi.w, lo.w);
          const int t = c0 + j8;                      // token within this warp's half: block t >> 6, chunk (t & 63) >> 3
          if (head_ok) *reinterpret_cast<uint4 *>(p_row + (size_t)(t >> 6) * MP_QBLK + mp_swz(row16, (t & 63) >> 3)) = even ? hi : lo;
        }
      }
      tc_fence_before();
      if (lane < 16) xs_sum[c][row16] = sum;
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&s_free_bar));
        mbar_arrive(smem_u32(&p_ready_bar));
        mbar_arrive(smem_u32(&x_bar));
      }
      {
        bool ok = mbar_wait(smem_u32(&x_bar), (uint32_t)(2 * k + 1) & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      if (c == 0 && head_ok && even)
        part_ml[((size_t)r * max_splits + split) * n_heads + head] = make_float2(mx, xs_sum[0][row16] + xs_sum[1][row16]);
    }
  } else if (warp == 12 || warp == 13 || warp == 16 || warp == 17) {
    // ---------------- output accumulator -> the split's partial ----------------
    const int q = warp & 3, c = warp >= 16 ? 1 : 0;  // TMEM lane quarter, column half
    const int row16 = 16 * q + (lane & 15), head = row16 >> 1;
    const bool head_ok = lane < 16 && head < n_heads;
    const bool even = (lane & 1) == 0;
    const int CW = NH / 2;                           // columns of this warp (32, 64 or 128)
    const uint32_t o_lane = o_tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(c * CW);
    int n_o = 0;
    for (int it = item_lo; it < item_hi && !failed; ++it) {
      int r, split;
      locate(it, r, split);
      for (int half = 0; half < n_half && !failed; ++half, ++n_o) {
        bool ok = mbar_wait(smem_u32(&o_full_bar), (uint32_t)n_o & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
        tc_fence_after();
        // both lanes of a pair hold the sum of the hi and lo rows: the even one stores columns 0-15 of every 32, the odd one 16-31
        float *dst = part_o + (((size_t)r * max_splits + split) * n_heads + head) * d_c + half * NH + c * CW + (even ? 0 : 16);
        for (int c0 = 0; c0 < CW; c0 += 32) {
          uint32_t v[32];
          mp_tmem_ld32(o_lane + (uint32_t)c0, v);
          tmem_ld_wait();
          float o[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float a = __uint_as_float(v[j]), b = __uint_as_float(v[16 + j]);
            const float sa = a + __shfl_xor_sync(0xffffffffu, a, 1), sb = b + __shfl_xor_sync(0xffffffffu, b, 1);
            o[j] = even ? sa : sb;
          }
          if (head_ok) {
#pragma unroll
            for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4 *>(dst + c0 + j) = make_float4(o[j], o[j + 1], o[j + 2], o[j + 3]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&o_free_bar));
      }
    }
  }
  if (failed || abort_flag) {
    if (lane == 0) atomicCAS(status, 0, DEV_TIMEOUT_EPILOGUE);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land before the CTA retires
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) tmem_dealloc(tmem_base, MP_TMEM_COLS);
}

// One block per (row, head), one thread per four latent dims: the row's splits in ascending order -> o_lat (fp32
// [B][n_heads][d_c]) or, when that is null, a bf16 hi/lo pair laid out head-major [n_heads][rows_per_head][d_c].
__global__ void __launch_bounds__(128) mla_paged_combine_kernel(const float2 *__restrict__ part_ml, const float *__restrict__ part_o,
                                                                const int *__restrict__ ctx, const int *__restrict__ row_pos,
                                                                const int *__restrict__ row_active, int B, int n_heads, int d_c,
                                                                int max_blocks, int max_splits, float *__restrict__ o_lat,
                                                                __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo,
                                                                int rows_per_head) {
  griddep_launch_dependents();
  __shared__ float2 sml[128];                       // the splits' (max, sum) pairs, fetched in one round trip
  const int r = (int)blockIdx.x / n_heads, h = (int)blockIdx.x - r * n_heads;
  const int d = 4 * (int)threadIdx.x;
  griddep_wait();                                   // before the first read of anything another kernel of the step wrote
  int c = row_pos ? (row_active[r] ? row_pos[r] + 1 : 0) : ctx[r];
  if (c <= 0) return;                               // a padding row is left alone (the whole block returns)
  c = c > max_blocks * MP_PAGE ? max_blocks * MP_PAGE : c;
  int ns = (c + MP_T - 1) / MP_T;
  if (ns > max_splits) ns = max_splits;
  const float2 *ml = part_ml + (size_t)r * max_splits * n_heads + h;
  const bool staged = ns <= 128;
  if (staged) {
    for (int s = threadIdx.x; s < ns; s += blockDim.x) sml[s] = __ldcg(&ml[(size_t)s * n_heads]);
    __syncthreads();
  }
  if (d >= d_c) return;
  auto pair_of = [&](int s) { return staged ? sml[s] : __ldcg(&ml[(size_t)s * n_heads]); };
  float M = -CUDART_INF_F;
  for (int s = 0; s < ns; ++s) M = fmaxf(M, pair_of(s).x);
  float den = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float2 v = pair_of(s);
    den += exp2f(v.x - M) * v.y;
  }
  const float inv = 1.f / den;
  const float *po = part_o + ((size_t)r * max_splits * n_heads + h) * d_c + d;
  const size_t stride = (size_t)n_heads * d_c;
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < ns; s0 += 4) {              // four splits' loads in flight; the sums stay in ascending order
    float4 x[4];
    float w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (s0 + e < ns) {
        x[e] = __ldcg(reinterpret_cast<const float4 *>(po + (size_t)(s0 + e) * stride));
        w[e] = exp2f(pair_of(s0 + e).x - M);
      }
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (s0 + e < ns) {
        o.x = fmaf(w[e], x[e].x, o.x); o.y = fmaf(w[e], x[e].y, o.y); o.z = fmaf(w[e], x[e].z, o.z); o.w = fmaf(w[e], x[e].w, o.w);
      }
  }
  o = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
  if (o_lat) {
    *reinterpret_cast<float4 *>(o_lat + ((size_t)r * n_heads + h) * d_c + d) = o;
  } else {
    const size_t at = ((size_t)h * rows_per_head + r) * d_c + d;
    const float v[4] = {o.x, o.y, o.z, o.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      hi[e] = __float2bfloat16_rn(v[e]);
      lo[e] = __float2bfloat16_rn(v[e] - __bfloat162float(hi[e]));
    }
    *reinterpret_cast<uint2 *>(out_hi + at) = *reinterpret_cast<const uint2 *>(hi);
    *reinterpret_cast<uint2 *>(out_lo + at) = *reinterpret_cast<const uint2 *>(lo);
  }
}

}  // namespace
}  // namespace corun

namespace corun {

int mla_max_splits(int max_context) { return (max_context + MP_T - 1) / MP_T; }
long long mla_part_ml_floats(int R, int nh, int max_context) { return ((long long)R * mla_max_splits(max_context) * nh * 2 + 3) / 4 * 4; }
long long mla_part_o_floats(int R, int nh, int rank, int max_context) { return (long long)R * mla_max_splits(max_context) * nh * rank; }

int mla_encode_maps(CUtensorMap *tmC, CUtensorMap *tmV, const void *pool, long long pool_pages, int rank, int rope, int page_run) {
  if (pool_pages < 1 || pool_pages * MP_PAGE >= (1ll << 31) || (page_run != 1 && page_run != 4)) return CORUN_EINVAL;
  const int bph = rank > 256 ? 4 : rank / 64;
  if (page_run == 4) {
    // block-major runs of 64 tokens: [run][block of 64 dims][64 tokens][64 dims].  Score pass: the pool as rows of 64
    // halfs, one [64 x 64] box = a block of a run, 8 KiB of contiguous memory.  Output pass: one box fetches a run's
    // 64 tokens x (up to) 256 dims as [8 groups][blocks][8 tokens][64 dims], the layout of an MN-major MMA operand.
    if (pool_pages % 4) return CORUN_EINVAL;
    const unsigned long long runs = (unsigned long long)pool_pages / 4, nblk = (unsigned long long)(rank + rope + 63) / 64;
    if (runs * nblk * 64 >= (1ull << 31)) return CORUN_EINVAL;
    const unsigned long long d2[2] = {64, runs * nblk * 64}, s2[1] = {128};
    const unsigned b2[2] = {64, 64};
    int rc = tma_encode_fp16_nd(tmC, pool, 2, d2, s2, b2);
    if (rc != CORUN_OK) return rc;
    const unsigned long long d5[5] = {64, 8, nblk, 8, runs}, s5[4] = {128, 64 * 128, 8 * 128, nblk * 64 * 128};
    const unsigned b5[5] = {64, 8, (unsigned)bph, 8, 1};
    return tma_encode_fp16_nd(tmV, pool, 5, d5, s5, b5);
  }
  // the pool as rows of rank + rope halfs, fetched in [16 tokens x 64 dims] boxes (the rope box reads past the
  // row's end when rope < 64: those columns arrive as zeros)
  int rc = tma_encode_2d(tmC, pool, 1, (unsigned long long)pool_pages * MP_PAGE, rank + rope, MP_PAGE, 64);
  if (rc != CORUN_OK) return rc;
  // the latent part once more as [8-token group][token in group][block of 64 dims][64 dims]: one box fetches a page's
  // 16 tokens x (up to) 256 dims as [2 groups][blocks][8 tokens][64 dims], the layout of an MN-major MMA operand
  const unsigned long long row_bytes = (unsigned long long)(rank + rope) * 2;
  const unsigned long long dims[4] = {64, 8, (unsigned long long)(rank / 64), (unsigned long long)pool_pages * 2};
  const unsigned long long strides[3] = {row_bytes, 128, 8 * row_bytes};
  const unsigned box[4] = {64, 8, (unsigned)bph, 2};
  return tma_encode_fp16_4d(tmV, pool, dims, strides, box);
}

cudaError_t launch_mla_attention(const CUtensorMap &tmC, const CUtensorMap &tmV, const float *q_lat, long long q_row_stride,
                                 long long q_head_stride, const float *q_rope, const int *block_table, int max_blocks,
                                 const int *ctx, const Rows *rows, int R, const MlaDims &d, float scale, int max_splits,
                                 float2 *part_ml, float *part_o, float *o_lat, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                 int rows_per_head, int num_sms, int *d_status, bool pdl, cudaStream_t st, int page_run) {
  static bool prepared = false;                     // idempotent; a race only repeats it
  if (!prepared) {
    cudaError_t e = cudaFuncSetAttribute(mla_paged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MP_SMEM);
    if (e != cudaSuccess) return e;
    prepared = true;
  }
  const int *row_slot = rows ? rows->slot : nullptr, *row_pos = rows ? rows->pos : nullptr, *row_active = rows ? rows->active : nullptr;
  cudaError_t ce = launch_k(mla_paged_kernel, dim3(num_sms), dim3(MP_THREADS), MP_SMEM, st, pdl, tmC, tmV, q_lat, q_row_stride,
                            q_head_stride, q_rope, block_table, max_blocks, ctx, row_slot, row_pos, row_active, R, d.nh, d.rank, d.rope,
                            scale * 1.4426950408889634f, max_splits, part_ml, part_o, d_status, page_run);
  if (ce != cudaSuccess) return ce;
  return launch_k(mla_paged_combine_kernel, dim3(R * d.nh), dim3(128), 0, st, true, part_ml, part_o, ctx, row_pos, row_active, R, d.nh,
                  d.rank, max_blocks, max_splits, o_lat, out_hi, out_lo, rows_per_head);
}

}  // namespace corun

using namespace corun;

extern "C" {

int64_t corun_mla_workspace_floats(int32_t B, int32_t n_heads, int32_t d_latent, int32_t max_context) {
  if (B < 1 || n_heads < 1 || d_latent < 1 || max_context < 1) return 0;
  return 64 + mla_part_ml_floats(B, n_heads, max_context) + mla_part_o_floats(B, n_heads, d_latent, max_context);
}

int corun_mla_attend(const float *q_lat, const float *q_rope, const void *pool, int64_t pool_pages, const int32_t *block_table,
                     int32_t max_blocks, const int32_t *ctx, int32_t B, int32_t n_heads, int32_t d_latent, int32_t d_rope,
                     float scale, float *o_lat, float *ws, void *cuda_stream) {
  if (!q_lat || !q_rope || !pool || !block_table || !ctx || !o_lat || !ws || B < 1 || B > MP_MAXB || n_heads < 1 ||
      n_heads > MP_MAXH || (d_latent != 64 && d_latent != 128 && d_latent != 256 && d_latent != 512) || d_rope < 8 ||
      d_rope > 64 || d_rope % 8 || max_blocks < 1 || pool_pages < 1 || pool_pages * MP_PAGE >= (1ll << 31) || !(scale > 0.f))
    return CORUN_EINVAL;
  if (reinterpret_cast<uintptr_t>(pool) % 16 || reinterpret_cast<uintptr_t>(o_lat) % 16 || reinterpret_cast<uintptr_t>(ws) % 16 ||
      reinterpret_cast<uintptr_t>(q_lat) % 16 || reinterpret_cast<uintptr_t>(q_rope) % 16)
    return CORUN_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int dev = 0, sms = 0;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (ce != cudaSuccess || sms < 1) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  CUtensorMap tm, tv;
  int rc = mla_encode_maps(&tm, &tv, pool, pool_pages, d_latent, d_rope, 1);   // any block table: one page per box
  if (rc != CORUN_OK) return rc;
  const int max_splits = mla_max_splits(max_blocks * MP_PAGE);
  int *status = reinterpret_cast<int *>(ws);
  float2 *part_ml = reinterpret_cast<float2 *>(ws + 64);
  float *part_o = ws + 64 + mla_part_ml_floats(B, n_heads, max_blocks * MP_PAGE);
  const MlaDims dims{n_heads, d_latent, 0, d_rope, 0};
  ce = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (ce == cudaSuccess)
    ce = launch_mla_attention(tm, tv, q_lat, (long long)n_heads * d_latent, d_latent, q_rope, block_table, max_blocks, ctx, nullptr, B, dims,
                              scale, max_splits, part_ml, part_o, o_lat, nullptr, nullptr, 0, sms, status, false, st, 1);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return CORUN_OK;
}

int corun_mla_sync(const float *ws, void *cuda_stream) {
  if (!ws) return CORUN_EINVAL;
  int hs = 0;
  cudaError_t ce = cudaMemcpyAsync(&hs, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return hs ? CORUN_ETIMEOUT : CORUN_OK;
}

}  // extern "C"
