// Request-local split-KV paged attention for one query token per row.
//
// A CTA owns (row, kv head, split of 128 cached tokens = 8 pages).  One thread
// issues TMA tile loads for the split's K and V pages ([16 tokens x 64 dims]
// boxes, 128-byte swizzle, straight from the page pool through one tensor map)
// and each of the 4 warps consumes its own quarter (2 pages) as soon as its
// mbarrier completes.  Scores and weighted values run on the tensor cores
// (mma.sync m16n8k16, fp16 inputs, fp32 accumulate): the cached K/V are fp16
// exactly; the query rows and the softmax weights enter as an fp16 hi/lo pair
// (x = hi + lo, 22 significand bits) stacked in the 16 rows of the A operand:
// rows 0..G-1 hold hi of the G query heads of this kv head, rows 8..8+G-1
// their lo parts, so both halves land in the same thread and are added there.
//
// Invariance: the split size is fixed, the split count is a function of the
// row's own context length, each warp walks its pages in ascending order with
// an online softmax, the 4 warps are merged in ascending order and the splits
// are combined in ascending order by one owner.  Nothing depends on other rows.
#include <cuda_fp16.h>
#include <math_constants.h>

#include "launch.cuh"
#include "ops.cuh"
#include "ptx.cuh"

namespace corun {

namespace {

constexpr int ATT_THREADS = 128;
constexpr int ATT_PAGES = ATT_SPLIT / KV_BLOCK;   // 8 pages per split
constexpr int BOX_BYTES = KV_BLOCK * 128;         // one [16 x 64] fp16 box

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D += A(16x16, row) * B(16x8, col), fp16 inputs, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_half2(__half a, __half b) {
  return (uint32_t)__half_as_ushort(a) | ((uint32_t)__half_as_ushort(b) << 16);
}
// x = hi + lo with hi, lo fp16
__device__ __forceinline__ void split_half(float x, __half &hi, __half &lo) {
  hi = __float2half_rn(x);
  lo = __float2half_rn(x - __half2float(hi));
}
// byte offset of 16-byte chunk `chunk` of row `row` inside a 128-byte-swizzled [16 x 128 B] box
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS)
attn_split_kernel(const __grid_constant__ CUtensorMap tmKV, const float *__restrict__ q, Rows rows, int nq, int group,
                  KvLayout kv, int layer, int max_splits, const int *__restrict__ work, const int *__restrict__ n_work,
                  float *__restrict__ part_acc, float *__restrict__ part_ml, int *status) {
  constexpr int NBOX = HD / 64;                  // boxes per (page, head) tile
  constexpr int TILE_BYTES = NBOX * BOX_BYTES;   // K (or V) of one page and head
  constexpr int KSTEPS = HD / 16;                // k-steps of the score MMA
  constexpr int NT = HD / 8;                     // n-tiles of the value MMA
  griddep_launch_dependents();
  griddep_wait();                                // the item list and q come from earlier kernels
  // persistent CTAs walk the step's list of (row, split) items x kv heads with a fixed stride; the
  // list only decides which CTA computes an item, never how it is computed
  const int n_items = *n_work * kv.n_kv;
  if ((int)blockIdx.x >= n_items) return;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar[4];
  __shared__ int page_s[ATT_PAGES];
  __shared__ int abort_flag;
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;     // K tiles, then V tiles
  const uint32_t v_tiles = tiles + ATT_PAGES * TILE_BYTES;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    abort_flag = 0;
    for (int w = 0; w < 4; ++w) mbar_init(smem_u32(&bar[w]), 1);
    fence_mbar_init();
    fence_proxy_async();
  }
  bool failed = false;
  uint32_t parity = 0;                           // phase of this warp's barrier: flips each time it is armed
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
  const int wi = work[item / kv.n_kv], g = item % kv.n_kv;
  const int r = wi >> 8, split = wi & 255;
  const int ctx = rows.pos[r] + 1;               // the new token attends to itself too
  const int t0 = split * ATT_SPLIT;
  const int n_pages = min(ATT_PAGES, (ctx - t0 + KV_BLOCK - 1) / KV_BLOCK);
  __syncthreads();                               // the previous item's merge buffers (tile memory) are free
  if (tid < ATT_PAGES)
    page_s[tid] = tid < n_pages ? kv.block_table[(size_t)rows.slot[r] * kv.max_blocks + t0 / KV_BLOCK + tid] : 0;
  __syncthreads();
  if (tid == 0) {
    const uint64_t pol = l2_policy_evict_first();       // the cache is streamed once per step
    for (int w = 0; w < 4; ++w) {
      const int np = min(2, n_pages - 2 * w);
      if (np <= 0) break;
      const uint32_t b = smem_u32(&bar[w]);
      mbar_arrive_expect_tx(b, (uint32_t)(np * 2 * TILE_BYTES));
      for (int p = 2 * w; p < 2 * w + np; ++p) {
        // pool rows: (((layer * pool_blocks + page) * 2 + k|v) * n_kv + head) * 16 + token
        const long long base = ((long long)layer * kv.pool_blocks + page_s[p]) * 2;
        const int row_k = (int)(((base + 0) * kv.n_kv + g) * KV_BLOCK);
        const int row_v = (int)(((base + 1) * kv.n_kv + g) * KV_BLOCK);
#pragma unroll
        for (int x = 0; x < NBOX; ++x) {
          tma_load_2d(tiles + p * TILE_BYTES + x * BOX_BYTES, &tmKV, x * 64, row_k, b, pol);
          tma_load_2d(v_tiles + p * TILE_BYTES + x * BOX_BYTES, &tmKV, x * 64, row_v, b, pol);
        }
      }
    }
  }

  // ---- query rows as A fragments: rows 0..G-1 hi, rows 8..8+G-1 lo (raw q; the scale goes on the scores)
  const int qrow = lane >> 2;                    // fragment row of this lane (and of its +8 partner)
  const bool row_used = qrow < group;
  uint32_t qa[KSTEPS][4];
  {
    const float *qp = q + (size_t)r * nq * HD + (size_t)(g * group + (row_used ? qrow : 0)) * HD + (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
      if (row_used) {
        x0 = *reinterpret_cast<const float2 *>(qp + ks * 16);
        x1 = *reinterpret_cast<const float2 *>(qp + ks * 16 + 8);
      }
      __half h0, l0, h1, l1, h2, l2, h3, l3;
      split_half(x0.x, h0, l0); split_half(x0.y, h1, l1);
      split_half(x1.x, h2, l2); split_half(x1.y, h3, l3);
      qa[ks][0] = pack_half2(h0, h1);   // (row, k..k+1)      hi
      qa[ks][1] = pack_half2(l0, l1);   // (row + 8, k..k+1)  lo
      qa[ks][2] = pack_half2(h2, h3);   // (row, k+8..k+9)    hi
      qa[ks][3] = pack_half2(l2, l3);   // (row + 8, ...)     lo
    }
  }
  const float sscale = (HD == 128 ? 0.08838834764831845f : 0.125f) * 1.4426950408889634f;   // log2(e)/sqrt(hd)

  float o[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
  float m_run = -CUDART_INF_F, l_run = 0.f;

  const int warp_t0 = t0 + warp * 32;
  if (warp_t0 < ctx) {
    bool ok = mbar_wait(smem_u32(&bar[warp]), parity, &abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    parity ^= 1u;                                // armed exactly when this warp has tokens (warp_t0 < ctx)
    if (!ok) {
      failed = true;
    } else {
      // ldmatrix lane roles: matrix mi = lane / 8, row inside it = lane % 8
      const int mi = lane >> 3, mr = lane & 7;
      for (int step = 0; step < 2; ++step) {
        const int p = warp * 2 + step;
        const int tok0 = t0 + p * KV_BLOCK;
        if (tok0 >= ctx) break;                                   // warp-uniform
        const uint32_t kt = tiles + p * TILE_BYTES, vt = v_tiles + p * TILE_BYTES;
        // ---- scores S[16 x 16 tokens]: two n-tiles of 8 tokens
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          // matrices: (tokens 0-7, dims lo), (tokens 0-7, dims hi), (tokens 8-15, dims lo), (tokens 8-15, dims hi)
          const int row = (mi >> 1) * 8 + mr;
          const int chunk = (ks & 3) * 2 + (mi & 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kt + (ks >> 2) * BOX_BYTES + swz(row, chunk), b0, b1, b2, b3);
          mma16816(s0, qa[ks], b0, b1);
          mma16816(s1, qa[ks], b2, b3);
        }
        // this lane: head `qrow`, tokens tok0 + (lane&3)*2 + {0,1} (n-tile 0) and + 8 (n-tile 1); hi + lo rows
        float sc[4];
        sc[0] = (s0[0] + s0[2]) * sscale; sc[1] = (s0[1] + s0[3]) * sscale;
        sc[2] = (s1[0] + s1[2]) * sscale; sc[3] = (s1[1] + s1[3]) * sscale;
        const int tk = tok0 + (lane & 3) * 2;
        if (tk >= ctx) sc[0] = -CUDART_INF_F;
        if (tk + 1 >= ctx) sc[1] = -CUDART_INF_F;
        if (tk + 8 >= ctx) sc[2] = -CUDART_INF_F;
        if (tk + 9 >= ctx) sc[3] = -CUDART_INF_F;
        float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));      // max over the 16 tokens of this row
        const float m_new = fmaxf(m_run, mx);                      // finite: token tok0 is valid
        const float alpha = exp2f(m_run - m_new);                  // 0 on the first step
        float pr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) pr[i] = exp2f(sc[i] - m_new);
        l_run = l_run * alpha + ((pr[0] + pr[1]) + (pr[2] + pr[3]));   // this lane's tokens; lanes are added at the end
        m_run = m_new;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          o[nt][0] *= alpha; o[nt][1] *= alpha; o[nt][2] *= alpha; o[nt][3] *= alpha;
        }
        __half ph[4], pl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split_half(pr[i], ph[i], pl[i]);
        uint32_t pa[4];
        pa[0] = pack_half2(ph[0], ph[1]);   // (row, tokens 0-7 pair)      hi
        pa[1] = pack_half2(pl[0], pl[1]);   // (row + 8, ...)              lo
        pa[2] = pack_half2(ph[2], ph[3]);   // (row, tokens 8-15 pair)     hi
        pa[3] = pack_half2(pl[2], pl[3]);   // (row + 8, ...)              lo
        // ---- weighted values O[16 x HD] += P[16 x 16 tokens] * V[16 tokens x HD]
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
          // matrices: (tokens 0-7, dims d0..d0+7), (tokens 8-15, same dims), (tokens 0-7, d0+8..), (tokens 8-15, d0+8..)
          const int row = (mi & 1) * 8 + mr;
          const int chunk = ((np * 2) & 7) + (mi >> 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_trans(vt + ((np * 16) >> 6) * BOX_BYTES + swz(row, chunk), b0, b1, b2, b3);
          mma16816(o[2 * np], pa, b0, b1);
          mma16816(o[2 * np + 1], pa, b2, b3);
        }
      }
    }
  }
  // row sums: add the 4 lanes that share a fragment row (fixed order)
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);

  // ---- merge the 4 warps in ascending order (the tile memory is free once every warp is here)
  __syncthreads();
  float *o_s = reinterpret_cast<float *>(smem_raw + (tiles - smem_u32(smem_raw)));   // [4][8][HD]
  float *m_s = o_s + 4 * 8 * HD;                                                     // [4][8]
  float *l_s = m_s + 32;                                                             // [4][8]
  if (row_used) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int d = nt * 8 + (lane & 3) * 2;
      float2 v = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);   // hi rows + lo rows
      *reinterpret_cast<float2 *>(&o_s[(warp * 8 + qrow) * HD + d]) = v;
    }
    if ((lane & 3) == 0) {
      m_s[warp * 8 + qrow] = m_run;
      l_s[warp * 8 + qrow] = l_run;
    }
  }
  __syncthreads();
  for (int idx = tid; idx < group * HD; idx += ATT_THREADS) {
    const int h = idx / HD, d = idx - h * HD;
    float M = m_s[h];
#pragma unroll
    for (int w = 1; w < 4; ++w) M = fmaxf(M, m_s[w * 8 + h]);     // warp 0 always holds a valid token
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float wgt = exp2f(m_s[w * 8 + h] - M);                 // 0 for a warp without tokens
      num = fmaf(o_s[(w * 8 + h) * HD + d], wgt, num);
      den = fmaf(l_s[w * 8 + h], wgt, den);
    }
    const size_t slot = ((size_t)r * nq + g * group + h) * max_splits + split;
    part_acc[slot * HD + d] = num;
    if (d == 0) {
      part_ml[slot * 2] = M;
      part_ml[slot * 2 + 1] = den;
    }
  }
  }   // items
  if (failed || abort_flag) {
    if (tid == 0) atomicCAS(status, 0, DEV_TIMEOUT_EPILOGUE);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land before the CTA retires
  }
}

// Combines the splits of each (row, head) in ascending split order: one CTA per (head, row),
// one thread per output dim.  Output: bf16 hi/lo pair for the O projection.
__global__ void __launch_bounds__(128)
attn_combine_kernel(Rows rows, int nq, int hd, int max_splits, const float *__restrict__ part_acc,
                    const float *__restrict__ part_ml, __nv_bfloat16 *__restrict__ out_hi,
                    __nv_bfloat16 *__restrict__ out_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int j = blockIdx.x, r = blockIdx.y, d = threadIdx.x;
  float o = 0.f;
  if (rows.active[r]) {
    const int nsplit = (rows.pos[r] + 1 + ATT_SPLIT - 1) / ATT_SPLIT;
    const float *ml = part_ml + ((size_t)r * nq + j) * max_splits * 2;
    const float *pa = part_acc + ((size_t)r * nq + j) * max_splits * hd + d;
    float M = ml[0];
    for (int s = 1; s < nsplit; ++s) M = fmaxf(M, ml[2 * s]);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < nsplit; ++s) {
      const float w = exp2f(ml[2 * s] - M);
      num = fmaf(pa[(size_t)s * hd], w, num);
      den = fmaf(ml[2 * s + 1], w, den);
    }
    o = num / den;
  }
  const __nv_bfloat16 a = __float2bfloat16_rn(o);
  const __nv_bfloat16 b = __float2bfloat16_rn(o - __bfloat162float(a));
  const size_t idx = (size_t)r * nq * hd + (size_t)j * hd + d;
  out_hi[idx] = a;
  out_lo[idx] = b;
}

// Lists the (row, split) items of the step: active rows in ascending order, splits ascending.
// One CTA; rows <= 256.  Entry = row << 8 | split.
__global__ void __launch_bounds__(256) attn_worklist_kernel(Rows rows, int *__restrict__ work, int *__restrict__ n_work) {
  griddep_launch_dependents();
  griddep_wait();
  __shared__ int cnt[256];
  const int r = threadIdx.x;
  const int mine = (r < rows.R && rows.active[r]) ? (rows.pos[r] + 1 + ATT_SPLIT - 1) / ATT_SPLIT : 0;
  cnt[r] = mine;
  __syncthreads();
  int before = 0;
  for (int i = 0; i < r; ++i) before += cnt[i];
  for (int s = 0; s < mine; ++s) work[before + s] = (r << 8) | s;
  if (r == 255) *n_work = before + mine;
}

template <int HD>
constexpr size_t att_smem_bytes() {
  return (size_t)2 * ATT_PAGES * (HD / 64) * BOX_BYTES + 1024;
}

}  // namespace

cudaError_t attention_prepare() {
  cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)att_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)att_smem_bytes<64>());
}

cudaError_t launch_attn_worklist(const Rows &rows, int *work, int *n_work, cudaStream_t st) {
  if (rows.R > 256) return cudaErrorInvalidValue;
  return launch_k(attn_worklist_kernel, dim3(1), dim3(256), 0, st, true, rows, work, n_work);
}

cudaError_t launch_attention(const CUtensorMap &tmKV, const float *q, const Rows &rows, int nq, const KvLayout &kv,
                             int layer, int max_splits, const int *work, const int *n_work, int grid_ctas,
                             float *part_acc, float *part_ml, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                             int *d_status, cudaStream_t st) {
  const int group = nq / kv.n_kv;
  if (group < 1 || group > 8 || max_splits > 256) return cudaErrorInvalidValue;
  const long long most = (long long)rows.R * max_splits * kv.n_kv;
  const int grid = (int)(most < grid_ctas ? most : grid_ctas);
  cudaError_t e;
  if (kv.hd == 128)
    e = launch_k(attn_split_kernel<128>, dim3(grid), dim3(ATT_THREADS), att_smem_bytes<128>(), st, true, tmKV, q, rows, nq,
                 group, kv, layer, max_splits, work, n_work, part_acc, part_ml, d_status);
  else if (kv.hd == 64)
    e = launch_k(attn_split_kernel<64>, dim3(grid), dim3(ATT_THREADS), att_smem_bytes<64>(), st, true, tmKV, q, rows, nq,
                 group, kv, layer, max_splits, work, n_work, part_acc, part_ml, d_status);
  else
    return cudaErrorInvalidValue;
  if (e != cudaSuccess) return e;
  return launch_k(attn_combine_kernel, dim3(nq, rows.R), dim3(kv.hd), 0, st, true, rows, nq, kv.hd, max_splits, part_acc,
                  part_ml, out_hi, out_lo);
}

}  // namespace corun
