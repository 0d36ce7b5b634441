// Causal attention of a prefill chunk: the chunk's rows are consecutive tokens of ONE request, so a tile of
// query rows shares every key / value tile it reads (the decode kernel reads them once per query row).
//
// One CTA per (tile of 128 / G consecutive tokens, kv head), G = query heads per kv head.  The 128 rows of
// the tile are the (token, head) pairs; row m = token m / G, head m % G.  The CTA walks the key blocks of
// 128 cached tokens (8 pages) from position 0 to the tile's last token twice:
//   pass 1  S = Q * K^T per block, running row maxima (the exact maximum of every row over its keys);
//   pass 2  S again, P = exp2(S - max) (causal mask: key position <= the row's own position), row sums,
//           O += P * V; at the end O / sum -> bf16 hi/lo for the O projection.
// Computing the scores twice buys a softmax against the true maximum with no rescaling of the running
// output; the keys come from L2 the second time.
// S[128 rows x 128 keys] = Q[128 x hd] * K^T on tcgen05.mma (M = 128, N = 128, fp16, Q as a hi/lo pair: two
// MMAs per k-slice), TMEM lane = row, so the softmax of a row is local to one thread; P goes to shared memory
// as fp16 (its values lie in [0, 1]); O[128 x hd] += P[128 x 128] * V[128 x hd], one MMA per page from the
// transposed value tiles.  Roles: warp 0 streams key and value tiles with TMA (keys through a ring of two,
// values through one buffer), warp 1 issues the MMAs, warps 2-5 own the rows.
//
// Every reduction has one fixed order (keys ascending) that depends on the row's own position only; the
// launch shape depends on the chunk size only.  All waits are bounded.
#include <cuda_fp16.h>
#include <math_constants.h>

#include "launch.cuh"
#include "ops.cuh"
#include "ptx.cuh"

namespace corun {

namespace {

constexpr int PF_THREADS = 192;
constexpr int PF_KEYS = 128;                        // keys per block
constexpr int PF_PAGES = PF_KEYS / KV_BLOCK;        // 8
constexpr int PF_NK = 2;                            // key ring depth

__device__ __forceinline__ uint32_t pf_swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

template <int HD>
struct PfLayout {
  static constexpr int NHALF = HD / 64;
  static constexpr int Q_BYTES = NHALF * 128 * 128;           // one of hi / lo: [half][128 rows x 128 B]
  static constexpr int P_BYTES = 2 * 128 * 128;               // [key half][128 rows x 128 B]
  static constexpr int K_BYTES = NHALF * PF_PAGES * KV_BLOCK * 128;   // [half][page][16 x 128 B]
  static constexpr int VT_BYTES = HD * KV_BLOCK * 2;          // one page: [hd x 32 B]
  static constexpr int V_BYTES = PF_PAGES * VT_BYTES;
  // the value MMA reads hd rows of V^T as its N operand; nothing runs past the tile
  static constexpr size_t SMEM = (size_t)2 * Q_BYTES + P_BYTES + PF_NK * K_BYTES + V_BYTES + 1024;
};

template <int HD, int GROUP>
__global__ void __launch_bounds__(PF_THREADS, 1)
attn_prefill_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const float *__restrict__ q, Rows rows, int nq, KvLayout kv, __nv_bfloat16 *__restrict__ out_hi,
                    __nv_bfloat16 *__restrict__ out_lo, int *status) {
  using L = PfLayout<HD>;
  constexpr int TPT = 128 / GROUP;                  // tokens per tile
  constexpr int KSTEPS = HD / 16;
  griddep_launch_dependents();
  griddep_wait();                                   // q and the chunk's own keys / values come from the kernel before
  const int tile = blockIdx.x, g = blockIdx.y;
  const int row0 = tile * TPT;                      // first chunk row of the tile
  // the tile's last active row decides how many key blocks there are
  int last = -1;
  for (int t = min(TPT, rows.R - row0) - 1; t >= 0; --t)
    if (rows.active[row0 + t]) { last = t; break; }
  if (last < 0) return;                             // padding only (the same decision in every thread)
  const int n_blocks = rows.pos[row0 + last] / PF_KEYS + 1;
  const int slot = rows.slot[row0];

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t kfull[PF_NK], kempty[PF_NK], vfull, vempty, s_full, s_free, p_full, o_done;
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
    mbar_init(smem_u32(&vfull), 1); mbar_init(smem_u32(&vempty), 1);
    mbar_init(smem_u32(&s_full), 1);                // scores of a block are in TMEM (MMA -> rows)
    mbar_init(smem_u32(&s_free), 128);              // every row has read its scores (rows -> MMA)
    mbar_init(smem_u32(&p_full), 128);              // every row has written its weights (rows -> MMA)
    mbar_init(smem_u32(&o_done), 1);                // all value MMAs have completed (MMA -> rows)
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_s), 256);        // 128 columns of scores + up to 128 of output
    tmem_relinquish();
  }
  if (warp >= 2) {
    // ---- the query tile: row m = (token m / G, head m % G) as fp16 hi and lo tiles (q = hi + lo)
    const int m = tid - 64;
    const int t = m / GROUP, h = m % GROUP;
    const bool real = row0 + t < rows.R;
    const float *qr = q + ((size_t)(real ? row0 + t : row0) * nq + (size_t)g * GROUP + h) * HD;
#pragma unroll 4
    for (int d = 0; d < HD; d += 8) {
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
  const uint32_t s_tmem = tmem_base, o_tmem = tmem_base + 128;
  // fp16 x fp16 -> fp32, K-major operands; N at bit 17 (>> 3), M = 128 at bit 24 (>> 4)
  const uint32_t idesc_s = (1u << 4) | ((uint32_t)(PF_KEYS >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  const uint32_t idesc_o = (1u << 4) | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  bool failed = false;

  // pages of key block b that exist for this tile (the last block may be partial)
  const int ctx_tile = rows.pos[row0 + last] + 1;
  auto pages_of = [&](int b) { return min(PF_PAGES, (ctx_tile - b * PF_KEYS + KV_BLOCK - 1) / KV_BLOCK); };

  if (warp == 0) {
    // ---------------- producer: keys of every block twice (pass 1, pass 2), values once; one lane per page
    const uint64_t pol = l2_policy_evict_last();    // the tiles of the same request read the same cache rows
    for (int it = 0; it < 2 * n_blocks; ++it) {
      const int b = it % n_blocks, kbuf = it % PF_NK;
      const int n_pages = pages_of(b);
      if (it >= PF_NK) {
        bool ok = mbar_wait(smem_u32(&kempty[kbuf]), (uint32_t)(it / PF_NK - 1) & 1u, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { failed = true; break; }
      }
      const uint32_t fb = smem_u32(&kfull[kbuf]);
      if (lane == 0) mbar_arrive_expect_tx(fb, (uint32_t)(n_pages * L::NHALF * KV_BLOCK * 128));
      __syncwarp();
      int page = 0;
      if (lane < n_pages) {
        page = kv.block_table[(size_t)slot * kv.max_blocks + b * PF_PAGES + lane];
        const int row_k = (page * 2 * kv.n_kv + g) * KV_BLOCK;
#pragma unroll
        for (int x = 0; x < L::NHALF; ++x)
          tma_load_2d(k_ring + (uint32_t)kbuf * L::K_BYTES + (uint32_t)(x * PF_PAGES + lane) * (KV_BLOCK * 128), &tmK,
                      x * 64, row_k, fb, pol);
      }
      if (it >= n_blocks) {                         // pass 2: the block's values as well
        const int j = it - n_blocks;
        if (j >= 1) {
          bool ok = mbar_wait(smem_u32(&vempty), (uint32_t)(j - 1) & 1u, &abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { failed = true; break; }
        }
        const uint32_t fv = smem_u32(&vfull);
        if (lane == 0) mbar_arrive_expect_tx(fv, (uint32_t)(n_pages * L::VT_BYTES));
        __syncwarp();
        if (lane < n_pages) {
          const int row_v = (page * 2 * kv.n_kv + kv.n_kv + g) * HD;
          tma_load_2d(v_buf + (uint32_t)lane * L::VT_BYTES, &tmV, 0, row_v, fv, pol);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      for (int it = 0; it < 2 * n_blocks && !failed; ++it) {
        const int b = it % n_blocks, kbuf = it % PF_NK;
        const bool pass2 = it >= n_blocks;
        // the rows must have read the previous block's scores before they are overwritten
        if (it >= 1 && !mbar_wait(smem_u32(&s_free), (uint32_t)(it - 1) & 1u, &abort_flag)) { failed = true; break; }
        if (!mbar_wait(smem_u32(&kfull[kbuf]), (uint32_t)(it / PF_NK) & 1u, &abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t kt = k_ring + (uint32_t)kbuf * L::K_BYTES;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const uint64_t adv = (uint64_t)((ks & 3) * 2);
          const uint64_t bk = umma_desc_sw128(kt + (uint32_t)(ks >> 2) * (PF_PAGES * KV_BLOCK * 128)) + adv;
          const uint64_t ah = umma_desc_sw128(q_hi + (uint32_t)(ks >> 2) * (128 * 128)) + adv;
          const uint64_t al = umma_desc_sw128(q_lo + (uint32_t)(ks >> 2) * (128 * 128)) + adv;
          umma_bf16(s_tmem, ah, bk, idesc_s, ks > 0 ? 1u : 0u);    // operand format (fp16) is in idesc
          umma_bf16(s_tmem, al, bk, idesc_s, 1u);
        }
        umma_commit(smem_u32(&kempty[kbuf]));       // the key buffer is free once these MMAs have read it
        umma_commit(smem_u32(&s_full));
        if (pass2) {
          const int j = it - n_blocks;
          // O += P * V once the rows have written the block's weights and the values have landed
          if (!mbar_wait(smem_u32(&p_full), (uint32_t)j & 1u, &abort_flag)) { failed = true; break; }
          if (!mbar_wait(smem_u32(&vfull), (uint32_t)j & 1u, &abort_flag)) { failed = true; break; }
          tc_fence_after();
          const int n_pages = pages_of(b);
          for (int p = 0; p < n_pages; ++p) {
            const uint64_t a = umma_desc_sw128(p_tile + (uint32_t)(p >> 2) * (128 * 128)) + (uint64_t)((p & 3) * 2);
            const uint64_t bv = umma_desc_sw32(v_buf + (uint32_t)p * L::VT_BYTES);
            umma_bf16(o_tmem, a, bv, idesc_o, (j > 0 || p > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&vempty));           // the value buffer and the weight tile are free
        }
      }
      umma_commit(smem_u32(&o_done));               // arrives in any case: nobody may hang on it
    }
  } else {
    // ---------------- rows: thread m owns (token m / G, head m % G)
    const int quad = warp & 3;                      // the TMEM lane quarter this warp may read
    const int tl = quad * 32 + lane;                // TMEM lane = tile row of this thread
    const int t = tl / GROUP, h = tl % GROUP;
    const bool in_chunk = row0 + t < rows.R;
    const bool real = in_chunk && rows.active[in_chunk ? row0 + t : row0] != 0;
    const int pos = real ? rows.pos[row0 + t] : -1;                  // keys 0..pos are visible to this row
    const float sscale = (HD == 128 ? 0.08838834764831845f : 0.125f) * 1.4426950408889634f;   // log2(e)/sqrt(hd)
    uint8_t *p_ptr = base_ptr + 2 * L::Q_BYTES;
    float mx = -CUDART_INF_F, sum = 0.f;
    for (int it = 0; it < 2 * n_blocks; ++it) {
      const int b = it % n_blocks;
      const bool pass2 = it >= n_blocks;
      bool ok = mbar_wait(smem_u32(&s_full), (uint32_t)it & 1u, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { failed = true; break; }
      tc_fence_after();
      if (pass2 && it > n_blocks) {
        // the weight tile is reused: the previous block's value MMAs must have read it
        bool okv = mbar_wait(smem_u32(&vempty), (uint32_t)(it - n_blocks - 1) & 1u, &abort_flag);
        okv = __all_sync(0xffffffffu, okv);
        if (!okv) { failed = true; break; }
      }
      const int key0 = b * PF_KEYS;
#pragma unroll
      for (int c0 = 0; c0 < PF_KEYS; c0 += 16) {
        uint32_t sv[16];
        tmem_ld16(s_tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, sv);
        tmem_ld_wait();
        if (!pass2) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (key0 + c0 + j <= pos) mx = fmaxf(mx, __uint_as_float(sv[j]) * sscale);
        } else {
          __half ph[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float p = key0 + c0 + j <= pos ? exp2f(__uint_as_float(sv[j]) * sscale - mx) : 0.f;
            sum += p;                               // keys in ascending order
            ph[j] = __float2half_rn(p);
          }
          // weights as the A operand of the value MMA: [key half][row][64 keys], 128-byte swizzle
          const uint32_t off = (uint32_t)(c0 >> 6) * (128 * 128);
          *reinterpret_cast<uint4 *>(p_ptr + off + pf_swz(tl, (c0 & 63) >> 3)) = *reinterpret_cast<const uint4 *>(&ph[0]);
          *reinterpret_cast<uint4 *>(p_ptr + off + pf_swz(tl, ((c0 & 63) >> 3) + 1)) = *reinterpret_cast<const uint4 *>(&ph[8]);
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&s_free));
      if (pass2) {
        fence_proxy_async();
        mbar_arrive(smem_u32(&p_full));
      }
    }
    // ---- output row: O / sum as a bf16 hi/lo pair
    {
      bool ok = failed ? false : mbar_wait(smem_u32(&o_done), 0u, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) failed = true;
      tc_fence_after();
      if (ok) {   // every lane takes part in the TMEM loads (they are warp-wide); only rows with a token store
        const float inv = real ? 1.f / sum : 0.f;
        const size_t o = ((size_t)(row0 + t) * nq + (size_t)g * GROUP + h) * HD;
#pragma unroll
        for (int c0 = 0; c0 < HD; c0 += 16) {
          uint32_t ov[16];
          tmem_ld16(o_tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, ov);
          tmem_ld_wait();
          __nv_bfloat16 hi[16], lo[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float y = __uint_as_float(ov[j]) * inv;
            hi[j] = __float2bfloat16_rn(y);
            lo[j] = __float2bfloat16_rn(y - __bfloat162float(hi[j]));
          }
          if (real) {
            *reinterpret_cast<uint4 *>(out_hi + o + c0) = *reinterpret_cast<const uint4 *>(&hi[0]);
            *reinterpret_cast<uint4 *>(out_hi + o + c0 + 8) = *reinterpret_cast<const uint4 *>(&hi[8]);
            *reinterpret_cast<uint4 *>(out_lo + o + c0) = *reinterpret_cast<const uint4 *>(&lo[0]);
            *reinterpret_cast<uint4 *>(out_lo + o + c0 + 8) = *reinterpret_cast<const uint4 *>(&lo[8]);
          }
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
  if (warp == 1) tmem_dealloc(tmem_base, 256);
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
  const dim3 grid((rows.R + tpt - 1) / tpt, kv.n_kv);
#define CORUN_PF_CASE(HD_, G_) \
  if (kv.hd == HD_ && group == G_) return pf_launch<HD_, G_>(grid, st, tmK, tmV, q, rows, nq, kv, out_hi, out_lo, d_status);
  CORUN_PF_CASE(128, 1) CORUN_PF_CASE(128, 2) CORUN_PF_CASE(128, 4) CORUN_PF_CASE(128, 8)
  CORUN_PF_CASE(64, 1) CORUN_PF_CASE(64, 2) CORUN_PF_CASE(64, 4) CORUN_PF_CASE(64, 8)
#undef CORUN_PF_CASE
  return cudaErrorInvalidValue;
}

}  // namespace corun
