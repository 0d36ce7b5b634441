// Request-local split-KV paged attention for one query token per row, on tcgen05.
//
// An item is (row, kv head, split of 128 cached tokens = 8 pages); the step's items are listed in that
// order and every CTA takes one contiguous stretch of the list (its two consumer groups one half each),
// so consecutive items of a group mostly share their query rows.  That covers the first 7/8 of the list; the rest is dealt out two items at a
// time through a counter, so that CTAs that got through their stretch sooner take more of it (which CTA
// computes an item has no influence on any value).  One persistent CTA per SM:
//   warp 0        streams the items' keys with TMA into a ring of 3 key buffers ([16 tokens x 64 dims]
//                 boxes, 128-byte swizzle), warp 1 their values into a ring of 3 value buffers (cached like
//                 the keys and fetched through the same kind of box: rows of 128 bytes, which the TMA unit
//                 moves four times as fast as the 32-byte rows of a transposed value tile), straight from
//                 the page pool.  A key buffer is free again as soon as the scores
//                 exist, a value buffer at the end of the item, so the key loads run ahead of the value
//                 loads and more bytes are in flight than with whole-item buffers;
//   2 groups of 4 warps take the items alternately.  Per item a group
//     1. writes the query rows as fp16 hi/lo pairs into a [16 x hd] operand tile (rows 0..G-1 hi of
//        the G query heads of this kv head, rows 8..8+G-1 their lo parts; q = hi + lo, 22 bits),
//     2. S^T[128 tokens x 16] = K[128 x hd] * Q^T       (tcgen05.mma, M = 128, N = 16, K = 16 per step)
//        -> TMEM lane = token, so each of the 128 threads owns one cached token,
//     3. softmax over the item: exact max and a fixed-order sum over the 128 tokens,
//        weights written as fp16 hi/lo rows of a [16 x 128 tokens] operand tile,
//     4. O^T[hd dims x 16] = V^T[hd x 128 tokens] * P^T  (one MMA per page; the token-major value tile is
//        its MN-major A operand), TMEM lane = dim,
//     5. adds the hi and lo columns and writes the split's partial (max, sum, O) to global memory;
// A second kernel, one warp per (row, query head), combines the splits' partials in ascending split order
// (attn_combine_kernel): as a kernel of its own the combines all run at once, where combiner warps inside the
// first kernel left a serial tail of several microseconds behind each CTA's last item.
// The cached K / V are fp16 exactly, accumulation is fp32.
//
// Invariance: the split size is fixed, the split count is a function of the row's own context
// length, every reduction inside an item has one fixed order, and the splits are combined in
// ascending order by one warp.  The work list only decides which CTA computes an item.
#include <cuda_fp16.h>
#include <math_constants.h>

#include "checks.cuh"
#include "launch.cuh"
#include "ops.cuh"
#include "ptx.cuh"

namespace corun {

namespace {

constexpr int ATT_NBUF = 3;                        // item buffers in the ring
constexpr int ATT_GROUPS = 2;                      // consumer groups of 4 warps
constexpr int ATT_SLOTS = 6;                       // barrier slots: a multiple of both
constexpr int ATT_THREADS = 64 + ATT_GROUPS * 128; // two producer warps + consumers
constexpr int ATT_PAGES = ATT_SPLIT / KV_BLOCK;    // 8 pages per split
constexpr int KBOX_BYTES = KV_BLOCK * 128;         // one [16 tokens x 64 dims] fp16 key box
constexpr int OPND_BYTES = 16 * 128;               // one [16 rows x 64 cols] fp16 half of a q / p operand tile
constexpr uint32_t ATT_TMEM_COLS = 64;             // per group: 16 columns of S^T and 16 of O^T

// byte offset of 16-byte chunk `chunk` of row `row` inside a 128-byte-swizzled tile of 128-byte rows
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// x = hi + lo with hi, lo fp16
__device__ __forceinline__ void split_half(float x, __half &hi, __half &lo) {
  hi = __float2half_rn(x);
  lo = __float2half_rn(x - __half2float(hi));
}

// Combines the splits of one (row, head) by one warp.  Lanes first hold one split each (max by
// butterfly, which is exact; the denominator by a fixed butterfly over at most 32 lanes, then
// ascending chunks of 32), then every lane owns hd/32 output dims and adds the splits' weighted
// partial outputs in ascending split order.  Output: bf16 hi/lo pair for the O projection.
// The partials may come from other SMs: they are read past the L1 cache.
template <int HD>
__device__ __forceinline__ void attn_combine_pair(int r, int j, int nsplit, int nq, int max_splits,
                                                  const float *__restrict__ part_acc, const float *__restrict__ part_ml,
                                                  __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo,
                                                  int lane) {
  constexpr int DPL = HD / 32;                   // dims per lane (4 or 2)
  float o[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[i] = 0.f;
  const float2 *ml = reinterpret_cast<const float2 *>(part_ml) + ((size_t)r * nq + j) * max_splits;
  const float *pa = part_acc + ((size_t)r * nq + j) * max_splits * HD + lane * DPL;
  auto load_acc = [&](int s) -> float4 {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (s < nsplit) {
      const float *p = pa + (size_t)s * HD;
      if (DPL == 4) a = __ldcg(reinterpret_cast<const float4 *>(p));
      else { const float2 t = __ldcg(reinterpret_cast<const float2 *>(p)); a.x = t.x; a.y = t.y; }
    }
    return a;
  };
  auto add_acc = [&](const float4 &a, float ws) {
    o[0] = fmaf(a.x, ws, o[0]); o[1] = fmaf(a.y, ws, o[1]);
    if (DPL == 4) { o[DPL - 2] = fmaf(a.z, ws, o[DPL - 2]); o[DPL - 1] = fmaf(a.w, ws, o[DPL - 1]); }
  };
  float den = 0.f;
  if (nsplit <= 64) {
    // usual case: the (max, sum) pairs of all splits sit in two registers per lane, and the first
    // sixteen partial outputs are requested before anything depends on them
    const float2 none = make_float2(-CUDART_INF_F, 0.f);
    const float2 v0 = lane < nsplit ? __ldcg(ml + lane) : none;
    const float2 v1 = 32 + lane < nsplit ? __ldcg(ml + 32 + lane) : none;
    float4 a[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) a[u] = load_acc(u);
    float M = fmaxf(v0.x, v1.x);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, k));
    const float w0 = exp2f(v0.x - M), w1 = exp2f(v1.x - M);   // 0 beyond the last split
    float d0 = v0.y * w0, d1 = v1.y * w1;
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) {
      d0 += __shfl_xor_sync(0xffffffffu, d0, k);
      d1 += __shfl_xor_sync(0xffffffffu, d1, k);
    }
    den = nsplit > 32 ? d0 + d1 : d0;
    for (int sb = 0; sb < nsplit; sb += 16) {
      if (sb > 0) {
#pragma unroll
        for (int u = 0; u < 16; ++u) a[u] = load_acc(sb + u);
      }
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int sidx = sb + u;
        const float ws = __shfl_sync(0xffffffffu, sidx < 32 ? w0 : w1, sidx & 31);
        add_acc(a[u], ws);                         // beyond the last split: 0 * 0
      }
    }
  } else {
    float M = -CUDART_INF_F;
    for (int s0 = 0; s0 < nsplit; s0 += 32) {
      float m = (s0 + lane < nsplit) ? __ldcg(ml + s0 + lane).x : -CUDART_INF_F;
#pragma unroll
      for (int k = 16; k > 0; k >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, k));
      M = fmaxf(M, m);
    }
    for (int s0 = 0; s0 < nsplit; s0 += 32) {
      float2 v = (s0 + lane < nsplit) ? __ldcg(ml + s0 + lane) : make_float2(-CUDART_INF_F, 0.f);
      const float w = exp2f(v.x - M);              // this lane's split weight (0 beyond the last split)
      float d = v.y * w;
#pragma unroll
      for (int k = 16; k > 0; k >>= 1) d += __shfl_xor_sync(0xffffffffu, d, k);
      den += d;
      const int cnt = min(32, nsplit - s0);
      for (int sb = 0; sb < cnt; sb += 8) {          // eight splits' partial outputs are fetched together
        float4 a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = sb + u < cnt ? load_acc(s0 + sb + u) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 8; ++u) add_acc(a[u], __shfl_sync(0xffffffffu, w, (sb + u) & 31));
      }
    }
  }
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[i] = o[i] / den;
  const size_t idx = (size_t)r * nq * HD + (size_t)j * HD + lane * DPL;
#pragma unroll
  for (int i = 0; i < DPL; ++i) {
    const __nv_bfloat16 a = __float2bfloat16_rn(o[i]);
    out_hi[idx + i] = a;
    out_lo[idx + i] = __float2bfloat16_rn(o[i] - __bfloat162float(a));
  }
}

template <int HD>
struct AttLayout {
  static constexpr int NHALF = HD / 64;                          // 64-dim halves of a key row
  static constexpr int PAGE_BYTES = NHALF * KBOX_BYTES;          // a page's keys: [8-token group][half][8 x 128 B]
  static constexpr int K_BYTES = ATT_PAGES * PAGE_BYTES;         // keys of an item: [page][group][half][8 x 128 B]
  static constexpr int V_BYTES = K_BYTES;                        // values of an item: the same arrangement
  static constexpr int ITEM_BYTES = K_BYTES + V_BYTES;
  static constexpr int Q_BYTES = NHALF * OPND_BYTES;             // [half][16 x 128 B]
  static constexpr int P_BYTES = 2 * OPND_BYTES;                 // 128 tokens = 2 halves of 64
  static constexpr int GROUP_BYTES = Q_BYTES + P_BYTES;
  // the value MMA always covers 128 dims (M = 128), i.e. two blocks of 64 dims 1 KiB apart: with hd = 64 the
  // second one is the page's second token group (results never used); the pad keeps every read inside the buffer
  static constexpr int PAD_BYTES = (HD < 128) ? ATT_PAGES * KBOX_BYTES + KBOX_BYTES : 0;
  static constexpr size_t SMEM = (size_t)ATT_NBUF * ITEM_BYTES + ATT_GROUPS * GROUP_BYTES + PAD_BYTES + 1024;
};

// WHOLE_PAIRS: the ablation that hands out whole (row, kv head) pairs (a separate instantiation, so that the
// kernel of the product is exactly the code it is without it).
// TRACED: the per-item globaltimer stamps (debug), likewise.
template <int HD, int GROUP, bool WHOLE_PAIRS, bool TRACED>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_split_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const float *__restrict__ q, Rows rows, int nq, KvLayout kv, int max_splits,
                  const int *__restrict__ work, const int *__restrict__ n_work, float *__restrict__ part_acc,
                  float *__restrict__ part_ml, int *__restrict__ pool_count, int *status,
                  unsigned long long *trace) {
  using L = AttLayout<HD>;
  // optional timeline (debug): per CTA and item (first 64): [key load issued, keys landed, group starts, released, scores done, weights written, values landed, output done]
#define ATRACE(k, i) do { if (TRACED && trace && (k) < 64) trace[((size_t)blockIdx.x * 64 + (k)) * 8 + (i)] = globaltimer_ns(); } while (0)
  constexpr int KSTEPS = HD / 16;
  griddep_launch_dependents();
  constexpr int group = GROUP;                   // query heads per kv head

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t kfull_bar[ATT_SLOTS], vfull_bar[ATT_SLOTS];
  __shared__ __align__(8) uint64_t kempty_bar[ATT_NBUF], vempty_bar[ATT_NBUF];
  __shared__ __align__(8) uint64_t mma_bar[ATT_GROUPS];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  __shared__ int stop_s[ATT_GROUPS];             // group-uniform copy of abort_flag, refreshed once per item
  __shared__ float red_s[ATT_GROUPS][4][8];      // cross-warp softmax reductions
  // pairs of pool items drawn by the key producer for the whole CTA: ring of 4, one barrier each
  __shared__ __align__(8) uint64_t pool_bar[4];
  __shared__ int pool_pair[4];
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    abort_flag = 0;
    for (int g = 0; g < ATT_GROUPS; ++g) { stop_s[g] = 0; mbar_init(smem_u32(&mma_bar[g]), 1); }
    for (int s = 0; s < ATT_SLOTS; ++s) { mbar_init(smem_u32(&kfull_bar[s]), 1); mbar_init(smem_u32(&vfull_bar[s]), 1); }
    for (int b = 0; b < ATT_NBUF; ++b) { mbar_init(smem_u32(&kempty_bar[b]), 1); mbar_init(smem_u32(&vempty_bar[b]), 1); }
    for (int b = 0; b < 4; ++b) mbar_init(smem_u32(&pool_bar[b]), 1);
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_base_s), ATT_TMEM_COLS);
    tmem_relinquish();
  } else if (warp >= 2 && warp < 2 + 4 * ATT_GROUPS) {
    // operand tiles start out as zeros: rows of unused heads are never written and must stay finite
    uint4 *z = reinterpret_cast<uint4 *>(ring_ptr + (size_t)ATT_NBUF * L::ITEM_BYTES);
    for (int i = tid - 64; i < ATT_GROUPS * L::GROUP_BYTES / 16; i += ATT_GROUPS * 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  // everything above touches nothing that another kernel writes: it runs while the kernels before this one drain
  griddep_wait();                                // the item list, q and the newest cache rows come from earlier kernels
  // (the inputs through after_wait: no load through them may be moved up across the wait)
  q = after_wait(q); work = after_wait(work); n_work = after_wait(n_work);
  rows.pos = after_wait(rows.pos); rows.active = after_wait(rows.active); rows.slot = after_wait(rows.slot);
  kv.block_table = after_wait(kv.block_table);
  const int n_total = *n_work;
  if (n_total <= 0) {                            // the same in every thread of the CTA
    if (warp == 0) tmem_dealloc(tmem_base, ATT_TMEM_COLS);
    return;
  }
  // this CTA's stretch of the item list, and where the shared pool begins
  const int n_pairs = WHOLE_PAIRS ? n_work[1] : 0;   // > 0: the ablation that hands out whole (row, kv head) pairs (see item_of)
  const int n_fixed = n_pairs > 0 ? 0 : (int)(((long long)n_total * 7 / 8) / gridDim.x);
  const int item_lo = (int)blockIdx.x * n_fixed, pool_lo = (int)gridDim.x * n_fixed;
  bool failed = false;
  // instruction descriptor: D fp32 (bits 4-5 = 1), A and B fp16 (0), K-major, N = 16 (N >> 3 at bit 17),
  // M = 128 (M >> 4 at bit 24)
  const uint32_t idesc = (1u << 4) | ((uint32_t)(16 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

  // Item of this CTA's k-th slot (every role walks the slots 0, 1, 2, ... with the same ring indices):
  // first the fixed stretch, then pairs drawn from the pool.  The key producer draws (draw = true, whole
  // warp) and publishes the pair; the other roles wait for it.  -1: no more work; -2: nothing in this slot.
  // Ablation mode (n_pairs > 0): no parallelism inside a (row, kv head) pair.  A CTA draws whole pairs from
  // the counter, one at a time, and walks each pair's splits in order (its two groups in turn); the table
  // behind the item count gives every pair's first item and split count.  The values are the same either way.
  const int *pair_tab = n_work + 2;
  int pair_j = -1, pair_c = 0;
  int wp_base = 0, wp_ns = 0, wp_start = 0;
  auto item_of = [&](int k, bool draw) -> int {
    if (WHOLE_PAIRS && n_pairs > 0) {
      while (wp_start >= 0 && k >= wp_base + wp_ns) {
        wp_base += wp_ns;
        ++pair_j;
        int c = 0;
        if (draw) {
          if (lane == 0) {
            c = atomicAdd(pool_count, 1);
            pool_pair[pair_j & 3] = c;
            mbar_arrive(smem_u32(&pool_bar[pair_j & 3]));
          }
          c = __shfl_sync(0xffffffffu, c, 0);
        } else {
          if (!mbar_wait(smem_u32(&pool_bar[pair_j & 3]), (uint32_t)(pair_j >> 2) & 1u, &abort_flag)) return -1;
          c = pool_pair[pair_j & 3];
        }
        if (c >= n_pairs) { wp_start = -1; break; }
        wp_start = __ldg(pair_tab + 2 * c);
        wp_ns = __ldg(pair_tab + 2 * c + 1);
      }
      return wp_start < 0 ? -1 : wp_start + (k - wp_base);
    }
    if (k < n_fixed)   // even slots walk the first half of the stretch (group 0), odd slots the second half (group 1)
      return item_lo + ((k & 1) ? ((n_fixed + 1) >> 1) + (k >> 1) : (k >> 1));
    const int j = (k - n_fixed) >> 1;
    if (j != pair_j) {
      if (draw) {
        int c = 0;
        if (lane == 0) {
          c = atomicAdd(pool_count, 1);
          pool_pair[j & 3] = c;
          mbar_arrive(smem_u32(&pool_bar[j & 3]));
        }
        pair_c = __shfl_sync(0xffffffffu, c, 0);
      } else {
        if (!mbar_wait(smem_u32(&pool_bar[j & 3]), (uint32_t)(j >> 2) & 1u, &abort_flag)) return -1;
        pair_c = pool_pair[j & 3];
      }
      pair_j = j;
    }
    if (pool_lo + pair_c * 2 >= n_total) return -1;
    const int it = pool_lo + pair_c * 2 + ((k - n_fixed) & 1);
    return it < n_total ? it : -2;
  };
  // shared memory: [key ring][value ring][operand tiles of the groups]
  const uint32_t vring = ring + (uint32_t)ATT_NBUF * L::K_BYTES;
  if (warp < 2) {
    // ---------------- producers: warp 0 keys, warp 1 values; one lane per page ----------------
    const bool is_v = warp == 1;
    // decode streams the cache once per step: nothing of it is worth keeping in L2
    const uint64_t pol = l2_policy_evict_first();
    uint64_t *full = is_v ? vfull_bar : kfull_bar, *empty = is_v ? vempty_bar : kempty_bar;
    for (int k = 0;; ++k) {
      const int item = item_of(k, !is_v);
      if (item == -1) break;
      if (item == -2) continue;
      const int buf = k % ATT_NBUF, slot = k % ATT_SLOTS;
      // where the item's pages are: looked up before the wait for the buffer (three dependent loads)
      const int wi = work[item];
      const int r = wi >> 16, g = (wi >> 8) & 255, split = wi & 255;
      const int ctx = rows.pos[r] + 1;
      const int t0 = split * ATT_SPLIT;
      const int n_pages = min(ATT_PAGES, (ctx - t0 + KV_BLOCK - 1) / KV_BLOCK);
      int page = lane < n_pages ? kv.block_table[(size_t)rows.slot[r] * kv.max_blocks + t0 / KV_BLOCK + lane] : 0;
#ifdef CORUN_CHECKED
      if (!check_item(r, rows.R, g, kv.n_kv, split, ctx, ATT_SPLIT) || !check_page(page, kv.pool_blocks)) {
        atomicCAS(status, 0, DEV_BAD_INDEX);       // the load goes to the reserved page 0 instead: nothing faults
        page = 0;
      }
#endif
      if (k >= ATT_NBUF) {                               // the buffer's previous item must have been released
        bool ok = mbar_wait(smem_u32(&empty[buf]), (uint32_t)(k / ATT_NBUF - 1) & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      const uint32_t fb = smem_u32(&full[slot]);
      if (lane == 0) {
        if (!is_v) ATRACE(k, 0);
        mbar_arrive_expect_tx(fb, (uint32_t)(n_pages * L::NHALF * KBOX_BYTES));
      }
      __syncwarp();
      if (lane < n_pages) {
        // this layer's pages as groups of eight rows of hd halfs: the key tile of (page, head) is the two groups from
        //   2 * (page * 2 * n_kv + head), its value tile 2 * n_kv groups further on.  ONE box per tile (the TMA unit
        //   is bound by the number of boxes: 99 cycles for a 2 KB box): [2 groups][halves of 64 dims][8 tokens][64 dims]
        if (is_v) {
          const int grp_v = 2 * (page * 2 * kv.n_kv + kv.n_kv + g);
          tma_load_4d(vring + (uint32_t)buf * L::V_BYTES + (uint32_t)lane * L::PAGE_BYTES, &tmV, 0, 0, 0, grp_v, fb, pol);
        } else {
          const int grp_k = 2 * (page * 2 * kv.n_kv + g);
          tma_load_4d(ring + (uint32_t)buf * L::K_BYTES + (uint32_t)lane * L::PAGE_BYTES, &tmK, 0, 0, 0, grp_k, fb, pol);
        }
      }
    }
  } else {
    // ---------------- consumers ----------------
    const int gi = (warp - 2) >> 2, gtid = (tid - 64) & 127;
    const int quad = warp & 3;                     // the TMEM lane quarter this warp may read
    const int tl = quad * 32 + lane;               // TMEM lane of this thread: token (scores) / dim (values)
    const float sscale = (HD == 128 ? 0.08838834764831845f : 0.125f) * 1.4426950408889634f;   // log2(e)/sqrt(hd)
    const uint32_t q_tile = ring + ATT_NBUF * L::ITEM_BYTES + (uint32_t)gi * L::GROUP_BYTES;
    const uint32_t p_tile = q_tile + L::Q_BYTES;
    uint8_t *q_ptr = ring_ptr + (size_t)ATT_NBUF * L::ITEM_BYTES + (size_t)gi * L::GROUP_BYTES;
    uint8_t *p_ptr = q_ptr + L::Q_BYTES;
    const uint32_t s_tmem = tmem_base + (uint32_t)gi * 32;       // S^T: 16 columns
    const uint32_t o_tmem = s_tmem + 16;                          // O^T: 16 columns
    const uint32_t mbar = smem_u32(&mma_bar[gi]);
    uint32_t mma_phase = 0, full_bits = 0;         // bit j: phase of the full barriers of this group's j-th slot
    constexpr int QPT = (GROUP * (HD / 2) + 127) / 128;   // float2 query values per thread
    float2 qreg[QPT];
    auto load_q = [&](int r_, int g_) {
#pragma unroll
      for (int i = 0; i < QPT; ++i) {
        const int idx = gtid + i * 128;
        if (idx < group * (HD / 2)) {
          const int h = idx / (HD / 2), d = (idx - h * (HD / 2)) * 2;
          qreg[i] = *reinterpret_cast<const float2 *>(q + (size_t)r_ * nq * HD + (size_t)(g_ * group + h) * HD + d);
        }
      }
    };
    int q_built = -1, q_loaded = -1;               // (row, kv head) keys of the operand tile / of qreg
    for (int k = gi;; k += ATT_GROUPS) {
      const int item = item_of(k, false);
      if (item < 0) break;
      const int buf = k % ATT_NBUF, slot = k % ATT_SLOTS, j = slot / ATT_GROUPS;
      const int wi = work[item];
      const int r = wi >> 16, g = (wi >> 8) & 255, split = wi & 255;
      const int ctx = rows.pos[r] + 1;               // the new token attends to itself too
      const int t0 = split * ATT_SPLIT;
      const int n_pages = min(ATT_PAGES, (ctx - t0 + KV_BLOCK - 1) / KV_BLOCK);
      const uint32_t k_tiles = ring + (uint32_t)buf * L::K_BYTES;
      const uint32_t v_tiles = vring + (uint32_t)buf * L::V_BYTES;

      if (gtid == 0) ATRACE(k, 2);
      // ---- 1. query operand tile: rows h (hi) and 8 + h (lo) of head g * group + h; the scale goes on the
      //         scores.  Rebuilt only when (row, kv head) changes; the values were normally fetched one
      //         item ahead (qreg), so no global latency sits here.
      if ((wi >> 8) != q_built) {
        if (q_loaded != (wi >> 8)) load_q(r, g);
#pragma unroll
        for (int i = 0; i < QPT; ++i) {
          const int idx = gtid + i * 128;
          if (idx < group * (HD / 2)) {
            const int h = idx / (HD / 2), d = (idx - h * (HD / 2)) * 2;
            __half h0, l0, h1, l1;
            split_half(qreg[i].x, h0, l0);
            split_half(qreg[i].y, h1, l1);
            const uint32_t off = (uint32_t)(d >> 6) * OPND_BYTES + (uint32_t)((d & 7) * 2);
            const int chunk = (d & 63) >> 3;
            *reinterpret_cast<__half2 *>(q_ptr + off + swz(h, chunk)) = __halves2half2(h0, h1);
            *reinterpret_cast<__half2 *>(q_ptr + off + swz(8 + h, chunk)) = __halves2half2(l0, l1);
          }
        }
        q_built = q_loaded = wi >> 8;
      }
      if (k + ATT_GROUPS < n_fixed) {   // fetch the next item's query values now if they differ
        const int nwi = work[item + 1];
        if ((nwi >> 8) != q_built) { load_q(nwi >> 16, (nwi >> 8) & 255); q_loaded = nwi >> 8; }
      }
      fence_proxy_async();                           // the MMA reads this tile through the async proxy
      if (gtid == 0) stop_s[gi] = abort_flag;
      asm volatile("bar.sync %0, 128;" ::"r"(1 + gi) : "memory");
      if (stop_s[gi]) break;                         // the same decision in all 4 warps of the group

      // ---- 2. S^T = K * Q^T, issued by one thread once the item has landed
      if (gtid == 0) {
        const bool ok = mbar_wait(smem_u32(&kfull_bar[slot]), (full_bits >> j) & 1u, &abort_flag);
        ATRACE(k, 1);
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < KSTEPS; ++ks) {
            const uint64_t adv = (uint64_t)((ks & 3) * 2);      // 16 dims = 32 bytes inside the swizzled row
            // the half's 8-token groups lie NHALF KiB apart (the halves of a group are neighbours)
            const uint64_t a = umma_desc_sw128_sbo(k_tiles + (uint32_t)(ks >> 2) * 1024u, (uint32_t)L::NHALF * 1024u) + adv;
            const uint64_t b = umma_desc_sw128(q_tile + (uint32_t)(ks >> 2) * OPND_BYTES) + adv;
            umma_bf16(s_tmem, a, b, idesc, ks > 0 ? 1u : 0u);   // operand format (fp16) is in idesc
          }
        }
        umma_commit(mbar);                           // also arrives if the wait gave up: nobody may hang here
      }
      {
        bool ok = mbar_wait(mbar, mma_phase, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        mma_phase ^= 1u;
        if (!ok) failed = true;
      }
      tc_fence_after();
      if (gtid == 0) { mbar_arrive(smem_u32(&kempty_bar[buf])); ATRACE(k, 4); }   // the scores exist: the key buffer is free

      // ---- 3. softmax over the item; this thread owns token t0 + tl
      uint32_t sv[16];
      tmem_ld16(s_tmem + ((uint32_t)(quad * 32) << 16), sv);
      tmem_ld_wait();
      const bool tok_ok = t0 + tl < ctx;
      float sc[GROUP];
#pragma unroll
      for (int h = 0; h < GROUP; ++h) {
        sc[h] = tok_ok ? (__uint_as_float(sv[h]) + __uint_as_float(sv[8 + h])) * sscale : -CUDART_INF_F;
        // the warp's maximum in one instruction, on the order-preserving integer image of the float (exact)
        const uint32_t u = __float_as_uint(sc[h]);
        const uint32_t km = __reduce_max_sync(0xffffffffu, (u & 0x80000000u) ? ~u : (u | 0x80000000u));
        const float m = __uint_as_float((km & 0x80000000u) ? (km ^ 0x80000000u) : ~km);
        if (lane == h) red_s[gi][quad][h] = m;
      }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + gi) : "memory");
      float pr[GROUP], mx[GROUP];
      float my_sum = 0.f;                            // lane h keeps the warp's sum of head h
#pragma unroll
      for (int h = 0; h < GROUP; ++h) {
        // exact maximum over the 128 tokens (token t0 is always valid, so it is finite for used heads)
        mx[h] = fmaxf(fmaxf(red_s[gi][0][h], red_s[gi][1][h]), fmaxf(red_s[gi][2][h], red_s[gi][3][h]));
        pr[h] = exp2f(sc[h] - mx[h]);                // 0 for masked tokens
        float s = pr[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);   // fixed butterfly
        if (lane == h) my_sum = s;
      }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + gi) : "memory");   // everyone has read the maxima
      if (lane < GROUP) red_s[gi][quad][lane] = my_sum;
      // weights as fp16 hi/lo into the [16 x 128 tokens] operand tile: rows h and 8 + h, column = token
      {
        const uint32_t off = (uint32_t)(tl >> 6) * OPND_BYTES + (uint32_t)((tl & 7) * 2);
        const int chunk = (tl & 63) >> 3;
#pragma unroll
        for (int h = 0; h < GROUP; ++h) {
          __half ph, pl;
          split_half(pr[h], ph, pl);
          *reinterpret_cast<__half *>(p_ptr + off + swz(h, chunk)) = ph;
          *reinterpret_cast<__half *>(p_ptr + off + swz(8 + h, chunk)) = pl;
        }
      }
      fence_proxy_async();
      tc_fence_before();
      asm volatile("bar.sync %0, 128;" ::"r"(1 + gi) : "memory");

      // ---- 4. O^T = V^T * P^T, one MMA per loaded page (16 tokens)
      if (gtid == 0) {
        ATRACE(k, 5);
        const bool ok = mbar_wait(smem_u32(&vfull_bar[slot]), (full_bits >> j) & 1u, &abort_flag);
        ATRACE(k, 6);
        tc_fence_after();
        for (int p = 0; ok && p < n_pages; ++p) {
          // A = V^T of the page: [128 dims x 16 tokens] read MN-major from the token-major tile (two blocks of
          // 64 dims 1 KiB apart, two groups of 8 tokens NHALF KiB apart)
          const uint64_t a = umma_desc_sw128_mn(v_tiles + (uint32_t)p * L::PAGE_BYTES, 1024u, (uint32_t)L::NHALF * 1024u);
          const uint64_t b = umma_desc_sw128(p_tile + (uint32_t)(p >> 2) * OPND_BYTES) + (uint64_t)((p & 3) * 2);
          umma_bf16(o_tmem, a, b, idesc | (1u << 15), p > 0 ? 1u : 0u);
        }
        umma_commit(mbar);                           // also arrives if the wait gave up
      }
      full_bits ^= 1u << j;
      {
        bool ok = mbar_wait(mbar, mma_phase, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        mma_phase ^= 1u;
        if (!ok) failed = true;
      }
      tc_fence_after();
      if (gtid == 0) { mbar_arrive(smem_u32(&vempty_bar[buf])); ATRACE(k, 7); }   // the value buffer is free

      // ---- 5. this thread owns output dim tl: add the hi and lo columns, write the partial
      if (quad * 32 < HD) {                          // warp-uniform: with hd = 64 only lanes 0-63 hold dims
        uint32_t ov[16];
        tmem_ld16(o_tmem + ((uint32_t)(quad * 32) << 16), ov);
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < GROUP; ++h) {
          const size_t pslot = ((size_t)r * nq + g * group + h) * max_splits + split;
          part_acc[pslot * HD + tl] = __uint_as_float(ov[h]) + __uint_as_float(ov[8 + h]);
        }
      }
#pragma unroll
      for (int h = 0; h < GROUP; ++h) {
        if (gtid == h) {                           // red_s holds the four warps' sums by now
          const size_t pslot = ((size_t)r * nq + g * group + h) * max_splits + split;
          part_ml[pslot * 2] = mx[h];
          part_ml[pslot * 2 + 1] = ((red_s[gi][0][h] + red_s[gi][1][h]) + red_s[gi][2][h]) + red_s[gi][3][h];
        }
      }
      tc_fence_before();
      asm volatile("bar.sync %0, 128;" ::"r"(1 + gi) : "memory");   // the group's TMEM and operand tiles are free
      if (gtid == 0) ATRACE(k, 3);
    }
    if (gtid == 0) ATRACE(63, gi);
  }
  if (failed || abort_flag) {
    if (lane == 0) atomicCAS(status, 0, DEV_TIMEOUT_EPILOGUE);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land before the CTA retires
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) tmem_dealloc(tmem_base, ATT_TMEM_COLS);
}

// Lists the items of the step: active rows ascending, kv heads ascending, splits ascending.
// One CTA; rows <= 256.  Entry = row << 16 | kv head << 8 | split.
// n_work[0] = number of items; n_work[1] = number of (row, kv head) pairs listed behind it as (first item,
// split count) when whole_pairs is set (the ablation without parallelism inside a pair), else 0.
__global__ void __launch_bounds__(256) attn_worklist_kernel(Rows rows, int n_kv, int *__restrict__ work,
                                                            int *__restrict__ n_work, int *__restrict__ pool_counts,
                                                            int n_pool_counts, int whole_pairs) {
  griddep_launch_dependents();
  griddep_wait();
  for (int i = threadIdx.x; i < n_pool_counts; i += 256) pool_counts[i] = 0;   // one pool counter per attention launch of the step
  __shared__ int cnt[256];
  const int r = threadIdx.x;
  const int mine = (r < rows.R && rows.active[r]) ? (rows.pos[r] + 1 + ATT_SPLIT - 1) / ATT_SPLIT : 0;
  cnt[r] = mine;
  __syncthreads();
  // every warp lists one row at a time
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int row = warp; row < rows.R; row += 8) {
    int before = 0;
    for (int i = lane; i < row; i += 32) before += cnt[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    const int ns = cnt[row];
    for (int i = lane; i < ns * n_kv; i += 32) work[before * n_kv + i] = (row << 16) | ((i / ns) << 8) | (i % ns);
    if (whole_pairs && ns > 0) {
      int rows_before = 0;                          // active rows before this one
      for (int i = lane; i < row; i += 32) rows_before += cnt[i] > 0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) rows_before += __shfl_xor_sync(0xffffffffu, rows_before, o);
      for (int g = lane; g < n_kv; g += 32) {
        n_work[2 + 2 * (rows_before * n_kv + g)] = before * n_kv + g * ns;
        n_work[3 + 2 * (rows_before * n_kv + g)] = ns;
      }
    }
  }
  if (r == 255) {
    int tot = 0, act = 0;
    for (int i = 0; i < 256; ++i) { tot += cnt[i]; act += cnt[i] > 0; }
    n_work[0] = tot * n_kv;
    n_work[1] = whole_pairs ? act * n_kv : 0;
  }
}

// One warp per (row, query head): adds the row's split partials in ascending split order -> bf16 hi/lo.
template <int HD>
__global__ void __launch_bounds__(128) attn_combine_kernel(Rows rows, int nq, int max_splits,
                                                           const float *__restrict__ part_acc,
                                                           const float *__restrict__ part_ml,
                                                           __nv_bfloat16 *__restrict__ out_hi,
                                                           __nv_bfloat16 *__restrict__ out_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int w = (int)blockIdx.x * 4 + ((int)threadIdx.x >> 5);
  if (w >= rows.R * nq) return;
  const int r = w / nq, j = w - r * nq;
  if (!rows.active[r]) return;                     // padding rows keep what they held
  const int ns = (rows.pos[r] + 1 + ATT_SPLIT - 1) / ATT_SPLIT;
  attn_combine_pair<HD>(r, j, ns, nq, max_splits, part_acc, part_ml, out_hi, out_lo, (int)threadIdx.x & 31);
}

}  // namespace

namespace {
template <int HD, int GROUP>
cudaError_t prepare_one() {
  cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<HD, GROUP, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)AttLayout<HD>::SMEM);
#ifdef CORUN_BUILD_DEBUG
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_split_kernel<HD, GROUP, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)AttLayout<HD>::SMEM);
#endif
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_split_kernel<HD, GROUP, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)AttLayout<HD>::SMEM);
  return e;
}
template <int HD>
cudaError_t launch_attn_split(int group, int grid, cudaStream_t st, const CUtensorMap &tmK, const CUtensorMap &tmV,
                         const float *q, const Rows &rows, int nq, const KvLayout &kv, int max_splits, const int *work,
                         const int *n_work, float *part_acc, float *part_ml, int *pool_count, int whole_pairs,
                         int *d_status, unsigned long long *trace) {
#ifdef CORUN_BUILD_DEBUG   // the stamped instantiation exists in debug builds only
#define CORUN_ATT_TRACED(G)                                                                                        \
    if (trace)                                                                                                     \
      return launch_k(attn_split_kernel<HD, G, false, true>, dim3(grid), dim3(ATT_THREADS), AttLayout<HD>::SMEM, st, true, tmK, tmV, q, \
                      rows, nq, kv, max_splits, work, n_work, part_acc, part_ml, pool_count, d_status, trace);
#else
#define CORUN_ATT_TRACED(G)
#endif
#define CORUN_ATT_CASE(G)                                                                                          \
  case G:                                                                                                          \
    if (whole_pairs)                                                                                               \
      return launch_k(attn_split_kernel<HD, G, true, false>, dim3(grid), dim3(ATT_THREADS), AttLayout<HD>::SMEM, st, true, tmK, tmV, q, \
                      rows, nq, kv, max_splits, work, n_work, part_acc, part_ml, pool_count, d_status, trace); \
    CORUN_ATT_TRACED(G)                                                                                            \
    return launch_k(attn_split_kernel<HD, G, false, false>, dim3(grid), dim3(ATT_THREADS), AttLayout<HD>::SMEM, st, true, tmK, tmV, q, \
                    rows, nq, kv, max_splits, work, n_work, part_acc, part_ml, pool_count, d_status, trace);
  switch (group) {
    CORUN_ATT_CASE(1)
    CORUN_ATT_CASE(2)
    CORUN_ATT_CASE(4)
    CORUN_ATT_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef CORUN_ATT_CASE
#undef CORUN_ATT_TRACED
}
}  // namespace

cudaError_t attention_prepare() {
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = prepare_one<128, 1>();
  if (e == cudaSuccess) e = prepare_one<128, 2>();
  if (e == cudaSuccess) e = prepare_one<128, 4>();
  if (e == cudaSuccess) e = prepare_one<128, 8>();
  if (e == cudaSuccess) e = prepare_one<64, 1>();
  if (e == cudaSuccess) e = prepare_one<64, 2>();
  if (e == cudaSuccess) e = prepare_one<64, 4>();
  if (e == cudaSuccess) e = prepare_one<64, 8>();
  return e;
}

cudaError_t launch_attn_worklist(const Rows &rows, int n_kv, int *work, int *n_work, int *pool_counts,
                                 int n_pool_counts, int whole_pairs, cudaStream_t st) {
  if (rows.R > 256 || n_kv > 255) return cudaErrorInvalidValue;
  return launch_k(attn_worklist_kernel, dim3(1), dim3(256), 0, st, true, rows, n_kv, work, n_work, pool_counts,
                  n_pool_counts, whole_pairs);
}

cudaError_t launch_attention(const CUtensorMap &tmK, const CUtensorMap &tmV, const float *q, const Rows &rows, int nq,
                             const KvLayout &kv, int layer, int max_splits, const int *work, const int *n_work,
                             int grid_ctas, float *part_acc, float *part_ml, int *pool_count,
                             __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int reuse, int *d_status, cudaStream_t st,
                             unsigned long long *trace) {
  (void)layer;   // the tensor maps are the layer's
  const int group = nq / kv.n_kv;
  if (group * kv.n_kv != nq || max_splits > 256) return cudaErrorInvalidValue;
  if (reuse == 1)   // a prefill chunk: consecutive tokens of one request
    return launch_attention_prefill(tmK, tmV, q, rows, nq, kv, out_hi, out_lo, d_status, st);
  const int whole_pairs = reuse == 2;   // the ablation: the item list carries the pair table
  const long long most = (long long)rows.R * max_splits * kv.n_kv;
  const int grid = (int)(most < grid_ctas ? most : grid_ctas);
  const int cgrid = (rows.R * nq + 3) / 4;
  cudaError_t ce = cudaErrorInvalidValue;
  if (kv.hd == 128) {
    ce = launch_attn_split<128>(group, grid, st, tmK, tmV, q, rows, nq, kv, max_splits, work, n_work, part_acc, part_ml,
                                pool_count, whole_pairs, d_status, trace);
    if (ce == cudaSuccess)
      ce = launch_k(attn_combine_kernel<128>, dim3(cgrid), dim3(128), 0, st, true, rows, nq, max_splits, part_acc, part_ml,
                    out_hi, out_lo);
  } else if (kv.hd == 64) {
    ce = launch_attn_split<64>(group, grid, st, tmK, tmV, q, rows, nq, kv, max_splits, work, n_work, part_acc, part_ml,
                               pool_count, whole_pairs, d_status, trace);
    if (ce == cudaSuccess)
      ce = launch_k(attn_combine_kernel<64>, dim3(cgrid), dim3(128), 0, st, true, rows, nq, max_splits, part_acc, part_ml,
                    out_hi, out_lo);
  }
  return ce;
}

}  // namespace corun
