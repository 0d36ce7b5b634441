// Causal attention of a prefill chunk: the chunk's rows are consecutive tokens of ONE request, so a tile of
// query rows shares every key / value tile it reads (the decode kernel reads them once per query row).
//
// One cluster of two CTAs per (tile of 128 / G consecutive tokens, kv head), G = query heads per kv head.
// The 128 rows of the tile are the (token, head) pairs; row m = token m / G, head m % G.  The key blocks of
// 128 cached tokens (8 pages) from position 0 to the tile's last token are dealt to the two CTAs in turn
// (even blocks to the first, odd ones to the second: more tiles in flight than one CTA's shared memory
// holds); each CTA produces the softmax of its own blocks (maximum, sum, unnormalised output), the second
// hands its three to the first through distributed shared memory and the first merges them, always as
// (first, second).  A CTA walks its blocks twice:
//   pass 1  S = Q * K^T per block, running row maxima (the exact maximum of every row over its keys);
//   pass 2  S again, P = exp2(S - max) (causal mask: key position <= the row's own position), row sums,
//           O += P * V; at the end O / sum -> bf16 hi/lo for the O projection.
// Computing the scores twice buys a softmax against the true maximum with no rescaling of the running
// output; the keys come from L2 the second time.
// S[128 rows x 128 keys] = Q[128 x hd] * K^T on tcgen05.mma (M = 128, N = 128, fp16, Q as a hi/lo pair: two
// MMAs per k-slice), TMEM lane = row, so the softmax of a row is local to one thread; P goes to shared memory
// as fp16 (its values lie in [0, 1]); O[128 x hd] += P[128 x 128] * V[128 x hd], one MMA per page with the
// token-major value tile as its MN-major B operand.  Roles: warp 0 streams the key tiles and warp 10 the value tiles with TMA (a ring of
// two each), warp 1 issues the MMAs, warps 2-9 own the rows: two threads per row, one for
// keys 0..63 and one for keys 64..127 of every block (two warps per scheduler hide each other's latencies);
// the two exchange their maxima after pass 1 and their sums at the end.  The scores and the weights
// are double-buffered: while the rows work on block j the tensor cores already compute the scores of block
// j + 1, and the value MMA of block j runs while the rows work on block j + 1.
//
// Every reduction has one fixed order (per thread: four interleaved partial sums over its keys in ascending
// order, then a fixed tree) that depends on the row's own position only; the
// launch shape depends on the chunk size only.  All waits are bounded.
#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include "launch.cuh"
#include "ops.cuh"
#include "ptx.cuh"

namespace corun {

namespace cg = cooperative_groups;

namespace {

constexpr int PF_THREADS = 352;
constexpr int PF_KEYS = 128;                        // keys per block
constexpr int PF_PAGES = PF_KEYS / KV_BLOCK;        // 8
constexpr int PF_NK = 2;                            // key ring depth
constexpr int PF_NV = 2;                            // value ring depth
constexpr int PF_KS = 2;                            // CTAs that share a tile's key blocks (the cluster size)

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pf_swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

template <int HD>
struct PfLayout {
  static constexpr int NHALF = HD / 64;
  static constexpr int Q_BYTES = NHALF * 128 * 128;           // one of hi / lo: [half][128 rows x 128 B]
  static constexpr int P_BYTES = 2 * 128 * 128;               // one weight tile: [key half][128 rows x 128 B]
  static constexpr int K_BYTES = NHALF * PF_PAGES * KV_BLOCK * 128;   // [half][page][16 x 128 B]
  static constexpr int VT_BYTES = NHALF * KV_BLOCK * 128;     // one page's values
  static constexpr int V_BYTES = PF_PAGES * VT_BYTES;         // [half][page][16 x 128 B], like the keys
  // the value MMA reads hd dims of V as its N operand (MN-major); nothing runs past the tile
  static constexpr size_t SMEM = (size_t)2 * Q_BYTES + P_BYTES + PF_NK * K_BYTES + PF_NV * V_BYTES + 1024;
};

template <int HD, int GROUP>
__global__ void __cluster_dims__(PF_KS, 1, 1) __launch_bounds__(PF_THREADS, 1)
attn_prefill_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const float *__restrict__ q, Rows rows, int nq, KvLayout kv, __nv_bfloat16 *__restrict__ out_hi,
                    __nv_bfloat16 *__restrict__ out_lo, int *status) {
  using L = PfLayout<HD>;
  constexpr int TPT = 128 / GROUP;                  // tokens per tile
  constexpr int KSTEPS = HD / 16;
  griddep_launch_dependents();
  griddep_wait();                                   // q and the chunk's own keys / values come from the kernel before
  const int tile = blockIdx.x / PF_KS, rank = blockIdx.x % PF_KS, g = blockIdx.y;
  const int row0 = tile * TPT;                      // first chunk row of the tile
  // the tile's last active row decides how many key blocks there are
  int last = -1;
  for (int t = min(TPT, rows.R - row0) - 1; t >= 0; --t)
    if (rows.active[row0 + t]) { last = t; break; }
  if (last < 0) return;                             // padding only (the same decision in the whole cluster)
  const int all_blocks = rows.pos[row0 + last] / PF_KEYS + 1;
  const int n_blocks = (all_blocks - rank + PF_KS - 1) / PF_KS;   // this CTA's blocks: rank, rank + PF_KS, ...
  auto blk = [&](int i) { return rank + i * PF_KS; };
  cg::cluster_group cluster = cg::this_cluster();
  const int slot = rows.slot[row0];

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t kfull[PF_NK], kempty[PF_NK], vfull[PF_NV], vempty[PF_NV], s_full[2], s_free[2], p_full,
      p_free, o_done;
  __shared__ float xch[2 * 128];                    // the maxima of the two threads of every row
  __shared__ __align__(8) uint64_t x_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_hi = base, q_lo = base + L::Q_BYTES, p_tile = q_lo + L::Q_BYTES, k_ring = p_tile + L::P_BYTES,
                 v_buf = k_ring + PF_NK * L::K_BYTES;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < PF_NK; ++i) { mbar_init(smem_u32(&kfull[i]), 1); mbar_init(smem_u32(&kempty[i]), 1); }
    for (int i = 0; i < PF_NV; ++i) { mbar_init(smem_u32(&vfull[i]), 1); mbar_init(smem_u32(&vempty[i]), 1); }
    mbar_init(smem_u32(&p_full), 256);              // every row thread has written its weights (rows -> MMA)
    mbar_init(smem_u32(&p_free), 1);                // the value MMAs have read the weight tile (MMA -> rows)
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&s_full[i]), 1);           // scores of a block are in TMEM (MMA -> rows)
      mbar_init(smem_u32(&s_free[i]), 256);         // every row thread has read its scores (rows -> MMA)
    }
    mbar_init(smem_u32(&o_done), 1);                // all value MMAs have completed (MMA -> rows)
    mbar_init(smem_u32(&x_bar), 256);               // both threads of every row have posted their value
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), 512);        // 2 x 128 columns of scores + up to 128 of output
    tmem_relinquish();
  }
  if (warp >= 2 && warp < 10) {
    // ---- the query tile: row m = (token m / G, head m % G) as fp16 hi and lo tiles (q = hi + lo)
    const int m = (tid - 64) & 127, dh = (tid - 64) >> 7;   // row, and which half of the head dimension
    const int t = m / GROUP, h = m % GROUP;
    const bool real = row0 + t < rows.R;
    const float *qr = q + ((size_t)(real ? row0 + t : row0) * nq + (size_t)g * GROUP + h) * HD;
#pragma unroll 4
    for (int d = dh * (HD / 2); d < (dh + 1) * (HD / 2); d += 8) {
      __half hi[8], lo[8];
#pragma unroll
      for (int j = 0; j < 8; j += 4) {
        const float4 v = real ? *reinterpret_cast<const float4 *>(qr + d + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          hi[j + i] = __float2half_rn(x[i]);
          lo[j + i] = __float2half_rn(x[i] - __half2float(hi[j + i]));
        }
      }
      const uint32_t off = (uint32_t)(d >> 6) * (128 * 128) + pf_swz(m, (d & 63) >> 3);
      *reinterpret_cast<uint4 *>(base_ptr + off) = *reinterpret_cast<const uint4 *>(hi);
      *reinterpret_cast<uint4 *>(base_ptr + L::Q_BYTES + off) = *reinterpret_cast<const uint4 *>(lo);
    }
    fence_proxy_async();                            // the MMAs read these tiles through the async proxy
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  const uint32_t s_tmem = tmem_base, o_tmem = tmem_base + 256;   // score buffer i at s_tmem + 128 i
  // fp16 x fp16 -> fp32, K-major operands; N at bit 17 (>> 3), M = 128 at bit 24 (>> 4)
  const uint32_t idesc_s = (1u << 4) | ((uint32_t)(PF_KEYS >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  const uint32_t idesc_o = (1u << 4) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);   // B (values) MN-major
  bool failed = false;

  // pages of key block b that exist for this tile (the last block may be partial)
  const int ctx_tile = rows.pos[row0 + last] + 1;
  auto pages_of = [&](int b) { return min(PF_PAGES, (ctx_tile - b * PF_KEYS + KV_BLOCK - 1) / KV_BLOCK); };

  // row threads: (tl, grp) owns (token tl / G, head tl % G), keys 64 grp .. 64 grp + 63 of every block
  const bool is_row = warp >= 2 && warp < 10;
  const int quad = warp & 3;                        // the TMEM lane quarter this warp may read
  const int grp = (warp - 2) >> 2;
  const int tl = quad * 32 + lane;                  // TMEM lane = tile row of this thread
  const int t = tl / GROUP, h = tl % GROUP;
  const bool in_chunk = row0 + t < rows.R;
  const bool real = is_row && in_chunk && rows.active[in_chunk ? row0 + t : row0] != 0;
  float mx = -CUDART_INF_F, l_own = 0.f;            // this CTA's maximum and sum of the row
  bool row_ok = false;                              // the row's part of this CTA's output is complete

  if (warp == 0 || warp == 10) {
    // ---------------- producers: warp 0 streams the keys of every block twice (pass 1, pass 2), warp 10 the
    // values once (pass 2); lane l fetches page l of a block, its page number read one step ahead of its use
    const uint64_t pol = l2_policy_evict_last();    // the tiles of the same request read the same cache rows
    const int *table = kv.block_table + (size_t)slot * kv.max_blocks;
    int page_next = (n_blocks > 0 && lane < pages_of(blk(0))) ? table[blk(0) * PF_PAGES + lane] : 0;
    if (warp == 0) {
      for (int it = 0; it < 2 * n_blocks; ++it) {
        const int b = blk(it % n_blocks), kbuf = it % PF_NK;
        const int n_pages = pages_of(b);
        const int page = page_next;
        {
          const int bn = blk((it + 1) % n_blocks);
          page_next = lane < pages_of(bn) ? table[bn * PF_PAGES + lane] : 0;
        }
        if (it >= PF_NK) {
          bool ok = mbar_wait(smem_u32(&kempty[kbuf]), (uint32_t)(it / PF_NK - 1) & 1u, &abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { failed = true; break; }
        }
        const uint32_t fb = smem_u32(&kfull[kbuf]);
        if (lane == 0) mbar_arrive_expect_tx(fb, (uint32_t)(n_pages * L::NHALF * KV_BLOCK * 128));
        __syncwarp();
        if (lane < n_pages) {
          const int row_k = (page * 2 * kv.n_kv + g) * KV_BLOCK;
#pragma unroll
          for (int x = 0; x < L::NHALF; ++x)
            tma_load_2d(k_ring + (uint32_t)kbuf * L::K_BYTES + (uint32_t)(x * PF_PAGES + lane) * (KV_BLOCK * 128), &tmK,
                        x * 64, row_k, fb, pol);
        }
      }
    } else {
      for (int j = 0; j < n_blocks; ++j) {
        const int vbuf = j % PF_NV;
        const int n_pages = pages_of(blk(j));
        const int page = page_next;
        if (j + 1 < n_blocks) page_next = lane < pages_of(blk(j + 1)) ? table[blk(j + 1) * PF_PAGES + lane] : 0;
        if (j >= PF_NV) {
          bool ok = mbar_wait(smem_u32(&vempty[vbuf]), (uint32_t)(j / PF_NV - 1) & 1u, &abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { failed = true; break; }
        }
        const uint32_t fv = smem_u32(&vfull[vbuf]);
        if (lane == 0) mbar_arrive_expect_tx(fv, (uint32_t)(n_pages * L::VT_BYTES));
        __syncwarp();
        if (lane < n_pages) {
          const int row_v = (page * 2 * kv.n_kv + kv.n_kv + g) * KV_BLOCK;
#pragma unroll
          for (int x = 0; x < L::NHALF; ++x)
            tma_load_2d(v_buf + (uint32_t)vbuf * L::V_BYTES + (uint32_t)(x * PF_PAGES + lane) * (KV_BLOCK * 128), &tmV, x * 64,
                        row_v, fv, pol);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: the scores of step `it`, then the value MMAs of the step before
    if (lane == 0) {
      auto issue_values = [&](int j) -> bool {      // O += P(j) * V(j)
        const int vbuf = j % PF_NV;
        if (!mbar_wait(smem_u32(&p_full), (uint32_t)j & 1u, &abort_flag)) return false;
        if (!mbar_wait(smem_u32(&vfull[vbuf]), (uint32_t)(j / PF_NV) & 1u, &abort_flag)) return false;
        tc_fence_after();
        const int n_pages = pages_of(blk(j));
        for (int p = 0; p < n_pages; ++p) {
          const uint64_t a = umma_desc_sw128(p_tile + (uint32_t)(p >> 2) * (128 * 128)) + (uint64_t)((p & 3) * 2);
          // B = the page's values [hd dims x 16 tokens], MN-major in the token-major tile: blocks of 64 dims a
          // tile half apart, groups of 8 tokens 1 KiB apart
          const uint64_t bv = umma_desc_sw128_mn(v_buf + (uint32_t)vbuf * L::V_BYTES + (uint32_t)p * (KV_BLOCK * 128),
                                                 PF_PAGES * KV_BLOCK * 128, 1024u);
          umma_bf16(o_tmem, a, bv, idesc_o, (j > 0 || p > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&vempty[vbuf]));       // the value buffer is free
        umma_commit(smem_u32(&p_free));             // and so is the weight tile
        return true;
      };
      for (int it = 0; it < 2 * n_blocks && !failed; ++it) {
        const int kbuf = it % PF_NK, sb = it & 1;
        // the rows must have read the scores of step it - 2 before their buffer is overwritten
        if (it >= 2 && !mbar_wait(smem_u32(&s_free[sb]), (uint32_t)((it >> 1) - 1) & 1u, &abort_flag)) { failed = true; break; }
        if (!mbar_wait(smem_u32(&kfull[kbuf]), (uint32_t)(it / PF_NK) & 1u, &abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t kt = k_ring + (uint32_t)kbuf * L::K_BYTES, st = s_tmem + (uint32_t)sb * 128;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const uint64_t adv = (uint64_t)((ks & 3) * 2);
          const uint64_t bk = umma_desc_sw128(kt + (uint32_t)(ks >> 2) * (PF_PAGES * KV_BLOCK * 128)) + adv;
          const uint64_t ah = umma_desc_sw128(q_hi + (uint32_t)(ks >> 2) * (128 * 128)) + adv;
          const uint64_t al = umma_desc_sw128(q_lo + (uint32_t)(ks >> 2) * (128 * 128)) + adv;
          umma_bf16(st, ah, bk, idesc_s, ks > 0 ? 1u : 0u);    // operand format (fp16) is in idesc
          umma_bf16(st, al, bk, idesc_s, 1u);
        }
        umma_commit(smem_u32(&kempty[kbuf]));       // the key buffer is free once these MMAs have read it
        umma_commit(smem_u32(&s_full[sb]));
        if (it > n_blocks && !issue_values(it - 1 - n_blocks)) { failed = true; break; }
      }
      if (!failed && n_blocks > 0 && !issue_values(n_blocks - 1)) failed = true;
      umma_commit(smem_u32(&o_done));               // arrives in any case: nobody may hang on it
    }
  } else if (warp < 10) {
    // ---------------- rows: threads (m, 0) and (m, 1) own (token m / G, head m % G), keys 64 grp .. 64 grp + 63
    const int pos = real ? rows.pos[row0 + t] : -1;                  // keys 0..pos are visible to this row
    const float sscale = (HD == 128 ? 0.08838834764831845f : 0.125f) * 1.4426950408889634f;   // log2(e)/sqrt(hd)
    uint8_t *p_ptr = base_ptr + 2 * L::Q_BYTES;
    const int c0 = grp * 64;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    // both threads of a row get both values; x: 2 x 128 floats of shared memory nobody else touches meanwhile
    auto exchange = [&](float *x, float mine, int phase, float &a, float &b2) -> bool {
      x[grp * 128 + tl] = mine;
      mbar_arrive(smem_u32(&x_bar));                // release: the store above is visible to who observes the phase
      bool ok = mbar_wait(smem_u32(&x_bar), (uint32_t)phase, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      a = x[tl];
      b2 = x[128 + tl];
      return ok;
    };
    for (int it = 0; it < 2 * n_blocks; ++it) {
      const int b = blk(it % n_blocks), sb = it & 1;
      const bool pass2 = it >= n_blocks;
      const int jb = it - n_blocks;                 // pass 2: the block's index among the value MMAs
      if (it == n_blocks) {                         // end of pass 1: the row's maximum over all its keys
        float m0, m1;
        if (!exchange(xch, mx, 0, m0, m1)) { failed = true; break; }
        mx = fmaxf(m0, m1);
      }
      bool ok = mbar_wait(smem_u32(&s_full[sb]), (uint32_t)(it >> 1) & 1u, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { failed = true; break; }
      tc_fence_after();
      const int key0 = b * PF_KEYS + c0;
      const bool masked = key0 + 63 > pos;          // only the row's last block (or padding) needs the mask
      const uint32_t st = s_tmem + (uint32_t)(sb * 128 + c0) + ((uint32_t)(quad * 32) << 16);
      uint8_t *pw = p_ptr + (size_t)grp * (128 * 128);
      uint32_t sv[4][16];
#pragma unroll
      for (int x = 0; x < 4; ++x) tmem_ld16(st + (uint32_t)(16 * x), sv[x]);
      tmem_ld_wait();
      if (!pass2) {
        if (!masked) {
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int j = 0; j < 16; ++j) mx = fmaxf(mx, __uint_as_float(sv[x][j]) * sscale);
        } else {
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (key0 + 16 * x + j <= pos) mx = fmaxf(mx, __uint_as_float(sv[x][j]) * sscale);
        }
      } else {
        __half2 ph[4][8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            float p0 = ex2_approx(fmaf(__uint_as_float(sv[x][j]), sscale, -mx));
            float p1 = ex2_approx(fmaf(__uint_as_float(sv[x][j + 1]), sscale, -mx));
            if (masked) {
              if (key0 + 16 * x + j > pos) p0 = 0.f;
              if (key0 + 16 * x + j + 1 > pos) p1 = 0.f;
            }
            acc[j & 3] += p0;
            acc[(j + 1) & 3] += p1;
            ph[x][j >> 1] = __floats2half2_rn(p0, p1);
          }
        }
        tc_fence_before();
        mbar_arrive(smem_u32(&s_free[sb]));         // the scores are in registers: their buffer may be overwritten
        if (jb >= 1) {
          // the weight tile is reused: the value MMAs of the block before must have read it
          bool okv = mbar_wait(smem_u32(&p_free), (uint32_t)(jb - 1) & 1u, &abort_flag);
          okv = __all_sync(0xffffffffu, okv);
          if (!okv) { failed = true; break; }
        }
        // weights as the A operand of the value MMA: [key half][row][64 keys], 128-byte swizzle
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          *reinterpret_cast<uint4 *>(pw + pf_swz(tl, 2 * x)) = *reinterpret_cast<const uint4 *>(&ph[x][0]);
          *reinterpret_cast<uint4 *>(pw + pf_swz(tl, 2 * x + 1)) = *reinterpret_cast<const uint4 *>(&ph[x][4]);
        }
      }
      if (pass2) {
        fence_proxy_async();
        mbar_arrive(smem_u32(&p_full));
      } else {
        tc_fence_before();
        mbar_arrive(smem_u32(&s_free[sb]));
      }
    }
    // ---- the row's sum in this CTA, and the end of the value MMAs
    if (n_blocks > 0) {
      float s0 = 0.f, s1 = 0.f;
      // the sums travel through the start of the query tile: this thread has seen the last scores arrive, so
      // every MMA that reads the queries has completed
      bool ok = !failed && exchange(reinterpret_cast<float *>(base_ptr), (acc[0] + acc[1]) + (acc[2] + acc[3]), 1, s0, s1);
      ok = ok && mbar_wait(smem_u32(&o_done), 0u, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) failed = true;
      tc_fence_after();
      l_own = s0 + s1;
      row_ok = ok;
    } else {
      row_ok = !failed;                             // no block of its own: maximum -inf, sum 0, output 0
    }
  }
  // ---------------- merge of the two CTAs' parts.  Every thread of both CTAs passes both cluster barriers.
  // After the first nobody reads its query or weight tiles any more; the second CTA then writes its output
  // (transposed: [column][row], so that a warp's stores are consecutive), maxima and sums into the first
  // CTA's query and weight tiles; after the second barrier the first CTA merges and stores.
  cluster.sync();
  if (is_row && rank != 0) {
    float *peer_o = reinterpret_cast<float *>(cluster.map_shared_rank(base_ptr, 0));
    float *peer_ml = reinterpret_cast<float *>(cluster.map_shared_rank(base_ptr + 2 * L::Q_BYTES, 0));
    const bool have = row_ok && n_blocks > 0;
#pragma unroll
    for (int d0 = grp * (HD / 2); d0 < (grp + 1) * (HD / 2); d0 += 16) {
      uint32_t ov[16];
      if (have) {                                   // warp-uniform: n_blocks and the outcome of the waits
        tmem_ld16(o_tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)d0, ov);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) ov[j] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) peer_o[(d0 + j) * 128 + tl] = __uint_as_float(ov[j]);
    }
    if (grp == 0) {
      peer_ml[tl] = have ? mx : -CUDART_INF_F;
      peer_ml[128 + tl] = have ? l_own : 0.f;
    }
  }
  cluster.sync();
  if (is_row && rank == 0) {
    // every lane takes part in the TMEM loads (they are warp-wide); only rows with a token store
    const float *o1 = reinterpret_cast<const float *>(base_ptr);
    const float *ml1 = reinterpret_cast<const float *>(base_ptr + 2 * L::Q_BYTES);
    if (row_ok) {
      const float m1 = ml1[tl], l1 = ml1[128 + tl];
      const float m = fmaxf(mx, m1);
      const float w0 = ex2_approx(mx - m), w1 = ex2_approx(m1 - m);   // the first CTA always has key 0: mx is finite
      const float inv = real ? 1.f / (l_own * w0 + l1 * w1) : 0.f;
      const float a0 = w0 * inv, a1 = w1 * inv;
      const size_t o = ((size_t)(row0 + t) * nq + (size_t)g * GROUP + h) * HD;
#pragma unroll
      for (int d0 = grp * (HD / 2); d0 < (grp + 1) * (HD / 2); d0 += 16) {
        uint32_t ov[16];
        tmem_ld16(o_tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)d0, ov);
        tmem_ld_wait();
        __nv_bfloat16 hi[16], lo[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float y = real ? __uint_as_float(ov[j]) * a0 + o1[(d0 + j) * 128 + tl] * a1 : 0.f;
          hi[j] = __float2bfloat16_rn(y);
          lo[j] = __float2bfloat16_rn(y - __bfloat162float(hi[j]));
        }
        if (real) {
          *reinterpret_cast<uint4 *>(out_hi + o + d0) = *reinterpret_cast<const uint4 *>(&hi[0]);
          *reinterpret_cast<uint4 *>(out_hi + o + d0 + 8) = *reinterpret_cast<const uint4 *>(&hi[8]);
          *reinterpret_cast<uint4 *>(out_lo + o + d0) = *reinterpret_cast<const uint4 *>(&lo[0]);
          *reinterpret_cast<uint4 *>(out_lo + o + d0 + 8) = *reinterpret_cast<const uint4 *>(&lo[8]);
        }
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
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

template <int HD, int GROUP>
cudaError_t pf_launch(dim3 grid, cudaStream_t st, const CUtensorMap &tmK, const CUtensorMap &tmV, const float *q,
                      const Rows &rows, int nq, const KvLayout &kv, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                      int *d_status) {
  static bool prepared = false;
  if (!prepared) {
    cudaError_t e = cudaFuncSetAttribute(attn_prefill_kernel<HD, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)PfLayout<HD>::SMEM);
    if (e != cudaSuccess) return e;
    prepared = true;
  }
  return launch_k(attn_prefill_kernel<HD, GROUP>, grid, dim3(PF_THREADS), PfLayout<HD>::SMEM, st, true, tmK, tmV, q, rows, nq,
                  kv, out_hi, out_lo, d_status);
}

}  // namespace

cudaError_t launch_attention_prefill(const CUtensorMap &tmK, const CUtensorMap &tmV, const float *q, const Rows &rows,
                                     int nq, const KvLayout &kv, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                                     int *d_status, cudaStream_t st) {
  const int group = nq / kv.n_kv;
  if (group * kv.n_kv != nq) return cudaErrorInvalidValue;
  if (group != 1 && group != 2 && group != 4 && group != 8) return cudaErrorInvalidValue;
  const int tpt = 128 / group;
  const dim3 grid(((rows.R + tpt - 1) / tpt) * PF_KS, kv.n_kv);
#define CORUN_PF_CASE(HD_, G_) \
  if (kv.hd == HD_ && group == G_) return pf_launch<HD_, G_>(grid, st, tmK, tmV, q, rows, nq, kv, out_hi, out_lo, d_status);
  CORUN_PF_CASE(128, 1) CORUN_PF_CASE(128, 2) CORUN_PF_CASE(128, 4) CORUN_PF_CASE(128, 8)
  CORUN_PF_CASE(64, 1) CORUN_PF_CASE(64, 2) CORUN_PF_CASE(64, 4) CORUN_PF_CASE(64, 8)
#undef CORUN_PF_CASE
  return cudaErrorInvalidValue;
}

}  // namespace corun
