// Multi-head latent attention at decode time in the absorbed form (see include/corun_mla.h).  Three kernels
// compute a row's partial (max, sum, output) per fixed-size piece of its cached tokens and a fourth combines
// the pieces in ascending order: mla_split_kernel (fp32 FMAs, 128-token splits), mla_split_mma_kernel
// (mma.sync, 128-token splits, staged then computed) and mla_chunk_mma_kernel (mma.sync, 512-token chunks
// streamed in 64-token tiles with an online softmax: the default).  Piece sizes are fixed and the piece count
// is a function of the row's own context: nothing depends on other rows.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include <cstdlib>

#include "../../include/corun_mla.h"
#include "gemm.cuh"

namespace {

constexpr int MLA_SPLIT = 128;      // cached tokens per split
constexpr int MLA_THREADS = 256;
constexpr int MLA_NH = 16;          // head slots of the shared-memory tiles (n_heads <= 16)

__global__ void __launch_bounds__(MLA_THREADS, 1)
mla_split_kernel(const float *__restrict__ q_lat, const float *__restrict__ q_rope, const __half *__restrict__ cache,
                 const int *__restrict__ ctx, int n_heads, int d_c, int d_r, int max_context, int max_splits, float scale,
                 float *__restrict__ part_o, float2 *__restrict__ part_ml) {
  const int s = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int n_ctx = min(ctx[b], max_context);   // a context beyond the cache is cut, never read
  const int t0 = s * MLA_SPLIT;
  if (t0 >= n_ctx) return;                           // the same decision in every thread
  const int n = min(MLA_SPLIT, n_ctx - t0);
  const int DK = d_c + d_r;
  const int pitch = DK + 2;                          // halfs; an odd number of 32-bit words: rows fall into different banks
  extern __shared__ __align__(16) unsigned char smem[];
  float *qs = reinterpret_cast<float *>(smem);                                   // [DK][16]: q[d][h]
  float *ps = qs + (size_t)DK * MLA_NH;                                          // [128][16]: scores, then weights
  float *red = ps + MLA_SPLIT * MLA_NH;                                          // [16] maxima, [16] sums
  __half *cs = reinterpret_cast<__half *>(red + 2 * MLA_NH);                     // [128][pitch]

  // ---- the row's absorbed queries (heads beyond n_heads: zeros)
  for (int i = tid; i < DK * MLA_NH; i += MLA_THREADS) {   // consecutive threads read consecutive d of one head
    const int h = i / DK, d = i - h * DK;
    float v = 0.f;
    if (h < n_heads) v = d < d_c ? q_lat[((size_t)b * n_heads + h) * d_c + d] : q_rope[((size_t)b * n_heads + h) * d_r + (d - d_c)];
    qs[d * MLA_NH + h] = v;
  }
  // ---- the split's cache rows (rows beyond the context: zeros): 16-byte loads, several in flight per thread
  {
    const int vecs = DK / 8;                         // uint4 per row (DK is a multiple of 8: rows are 16-byte aligned)
    const uint4 *src = reinterpret_cast<const uint4 *>(cache + ((size_t)b * max_context + t0) * DK);
    uint32_t *dst = reinterpret_cast<uint32_t *>(cs);
    const int total = MLA_SPLIT * vecs;
    for (int i0 = tid; i0 < total; i0 += MLA_THREADS * 6) {
      uint4 v[6];
#pragma unroll
      for (int k = 0; k < 6; ++k) {
        const int i = i0 + MLA_THREADS * k;
        const int t = i / vecs;
        v[k] = (i < total && t < n) ? src[i] : make_uint4(0u, 0u, 0u, 0u);   // rows are contiguous: src[t * vecs + j] = src[i]
      }
#pragma unroll
      for (int k = 0; k < 6; ++k) {
        const int i = i0 + MLA_THREADS * k;
        if (i < total) {
          const int t = i / vecs, j = i - t * vecs;
          uint32_t *d = dst + t * (pitch / 2) + 4 * j;
          d[0] = v[k].x; d[1] = v[k].y; d[2] = v[k].z; d[3] = v[k].w;
        }
      }
    }
  }
  __syncthreads();

  // ---- scores: thread = (tokens tp and tp + 64, heads 4 hq .. 4 hq + 3)
  {
    const int tp = tid & 63, hq = tid >> 6;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    const __half2 *c0 = reinterpret_cast<const __half2 *>(cs + (size_t)tp * pitch);
    const __half2 *c1 = reinterpret_cast<const __half2 *>(cs + (size_t)(tp + 64) * pitch);
#pragma unroll 4
    for (int d = 0; d < DK; d += 2) {
      const float2 a = __half22float2(c0[d >> 1]), e = __half22float2(c1[d >> 1]);
      const float4 qa = *reinterpret_cast<const float4 *>(qs + (size_t)d * MLA_NH + 4 * hq);
      const float4 qb = *reinterpret_cast<const float4 *>(qs + (size_t)(d + 1) * MLA_NH + 4 * hq);
      acc[0][0] = fmaf(a.x, qa.x, acc[0][0]); acc[0][1] = fmaf(a.x, qa.y, acc[0][1]);
      acc[0][2] = fmaf(a.x, qa.z, acc[0][2]); acc[0][3] = fmaf(a.x, qa.w, acc[0][3]);
      acc[0][0] = fmaf(a.y, qb.x, acc[0][0]); acc[0][1] = fmaf(a.y, qb.y, acc[0][1]);
      acc[0][2] = fmaf(a.y, qb.z, acc[0][2]); acc[0][3] = fmaf(a.y, qb.w, acc[0][3]);
      acc[1][0] = fmaf(e.x, qa.x, acc[1][0]); acc[1][1] = fmaf(e.x, qa.y, acc[1][1]);
      acc[1][2] = fmaf(e.x, qa.z, acc[1][2]); acc[1][3] = fmaf(e.x, qa.w, acc[1][3]);
      acc[1][0] = fmaf(e.y, qb.x, acc[1][0]); acc[1][1] = fmaf(e.y, qb.y, acc[1][1]);
      acc[1][2] = fmaf(e.y, qb.z, acc[1][2]); acc[1][3] = fmaf(e.y, qb.w, acc[1][3]);
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int t = tp + 64 * k;
#pragma unroll
      for (int j = 0; j < 4; ++j) ps[t * MLA_NH + 4 * hq + j] = t < n ? acc[k][j] * scale : -CUDART_INF_F;
    }
  }
  __syncthreads();

  // ---- softmax of the split per head: warp w takes heads 2 w and 2 w + 1; fixed orders throughout
  {
    const int warp = tid >> 5, lane = tid & 31;
    for (int h = 2 * warp; h < 2 * warp + 2; ++h) {
      float v[4], m = -CUDART_INF_F;
#pragma unroll
      for (int k = 0; k < 4; ++k) { v[k] = ps[(lane + 32 * k) * MLA_NH + h]; m = fmaxf(m, v[k]); }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      float l = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float p = expf(v[k] - m);             // exp(-inf) = 0 beyond the context
        ps[(lane + 32 * k) * MLA_NH + h] = p;
        l += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
      if (lane == 0) { red[h] = m; red[MLA_NH + h] = l; }
    }
  }
  __syncthreads();

  // ---- weighted latent sum: thread = dims (2 tid, 2 tid + 1) (+ 512 ...) of all heads, tokens ascending
  for (int d0 = 2 * tid; d0 < d_c; d0 += 2 * MLA_THREADS) {
    float acc[MLA_NH][2];
#pragma unroll
    for (int h = 0; h < MLA_NH; ++h) { acc[h][0] = 0.f; acc[h][1] = 0.f; }
#pragma unroll 2
    for (int t = 0; t < n; ++t) {
      const float2 c = __half22float2(*reinterpret_cast<const __half2 *>(cs + (size_t)t * pitch + d0));
      const float4 *p4 = reinterpret_cast<const float4 *>(ps + t * MLA_NH);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const float4 p = p4[g];
        acc[4 * g + 0][0] = fmaf(p.x, c.x, acc[4 * g + 0][0]); acc[4 * g + 0][1] = fmaf(p.x, c.y, acc[4 * g + 0][1]);
        acc[4 * g + 1][0] = fmaf(p.y, c.x, acc[4 * g + 1][0]); acc[4 * g + 1][1] = fmaf(p.y, c.y, acc[4 * g + 1][1]);
        acc[4 * g + 2][0] = fmaf(p.z, c.x, acc[4 * g + 2][0]); acc[4 * g + 2][1] = fmaf(p.z, c.y, acc[4 * g + 2][1]);
        acc[4 * g + 3][0] = fmaf(p.w, c.x, acc[4 * g + 3][0]); acc[4 * g + 3][1] = fmaf(p.w, c.y, acc[4 * g + 3][1]);
      }
    }
    for (int h = 0; h < n_heads; ++h)
      *reinterpret_cast<float2 *>(part_o + (((size_t)b * max_splits + s) * n_heads + h) * d_c + d0) = make_float2(acc[h][0], acc[h][1]);
  }
  if (tid < n_heads) part_ml[((size_t)b * max_splits + s) * n_heads + tid] = make_float2(red[tid], red[MLA_NH + tid]);
}

// ---------------------------------------------------------------- the same split on the warp-level tensor path
// mma.sync m16n8k16 (fp16 x fp16 -> fp32): the 16 heads are the M dimension of every instruction.  Queries and
// softmax weights enter as fp16 hi + lo pairs (two instructions per tile), the cache rows are fp16 as stored.
// Scores: warp w takes tokens 16 w .. 16 w + 15 (B operand = cache rows [token][dim], read with ldmatrix);
// weighted latent sum: warp w takes dims 64 w .. 64 w + 63 (B operand = the same rows read with ldmatrix.trans).
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void *p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t a) {   // a: shared-space byte address
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t a) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

constexpr int MLA_CP = 8;           // halfs of padding per cache / query row (rows stay 16-byte aligned, ldmatrix conflict-free)
constexpr int MLA_PP = 8;           // the same for the weight rows

__global__ void __launch_bounds__(MLA_THREADS, 1)
mla_split_mma_kernel(const float *__restrict__ q_lat, const float *__restrict__ q_rope, const __half *__restrict__ cache,
                     const int *__restrict__ ctx, int n_heads, int d_c, int d_r, int max_context, int max_splits, float scale,
                     float *__restrict__ part_o, float2 *__restrict__ part_ml) {
  const int s = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_ctx = min(ctx[b], max_context);   // a context beyond the cache is cut, never read
  const int t0 = s * MLA_SPLIT;
  if (t0 >= n_ctx) return;
  const int n = min(MLA_SPLIT, n_ctx - t0);
  const int DK = d_c + d_r;                          // a multiple of 16 (d_c % 64 == 0, d_r % 16 == 0 on this path)
  const int cp = DK + MLA_CP, pp = MLA_SPLIT + MLA_PP;
  extern __shared__ __align__(16) unsigned char smem[];
  __half *cs = reinterpret_cast<__half *>(smem);                     // [128][cp]   cache rows
  __half *qh = cs + (size_t)MLA_SPLIT * cp;                          // [16][cp]    query hi
  __half *ql = qh + (size_t)MLA_NH * cp;                             // [16][cp]    query lo
  __half *ph = ql + (size_t)MLA_NH * cp;                             // [16][pp]    weights hi
  __half *pl = ph + (size_t)MLA_NH * pp;                             // [16][pp]    weights lo
  float *sc = reinterpret_cast<float *>(pl + (size_t)MLA_NH * pp);   // [16][128]   scores
  float *red = sc + MLA_NH * MLA_SPLIT;                              // [16] maxima, [16] sums

  // ---- the split's cache rows straight into shared memory (cp.async: the whole tile in flight at once)
  {
    const int vecs = DK / 8;
    const __half *src = cache + ((size_t)b * max_context + t0) * DK;
    const int total = MLA_SPLIT * vecs;
    for (int i = tid; i < total; i += MLA_THREADS) {
      const int t = i / vecs, j = i - t * vecs;
      __half *d = cs + (size_t)t * cp + 8 * j;
      if (t < n) {
        const uint32_t da = (uint32_t)__cvta_generic_to_shared(d);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(da), "l"(src + (size_t)i * 8) : "memory");
      } else {
        *reinterpret_cast<uint4 *>(d) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  // ---- the row's absorbed queries as fp16 hi + lo (eight independent loads per thread in flight)
  for (int i0 = tid; i0 < DK * MLA_NH; i0 += MLA_THREADS * 8) {
    float v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int i = i0 + MLA_THREADS * k;
      const int h = i / DK, d = i - h * DK;
      v[k] = 0.f;
      if (i < DK * MLA_NH && h < n_heads)
        v[k] = d < d_c ? q_lat[((size_t)b * n_heads + h) * d_c + d] : q_rope[((size_t)b * n_heads + h) * d_r + (d - d_c)];
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int i = i0 + MLA_THREADS * k;
      if (i < DK * MLA_NH) {
        const int h = i / DK, d = i - h * DK;
        const __half hi = __float2half_rn(v[k]);
        qh[h * cp + d] = hi;
        ql[h * cp + d] = __float2half_rn(v[k] - __half2float(hi));
      }
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();

  // ---- scores S[16 heads][tokens 16 warp ..]: two n8 tiles per warp
  {
    float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
    const int tok0 = 16 * warp;
    // A (16 heads x 16 dims): lane -> row lane % 16, column block (lane / 16) * 8
    const __half *a_hi = qh + (size_t)(lane & 15) * cp + (lane >> 4) * 8;
    const __half *a_lo = ql + (size_t)(lane & 15) * cp + (lane >> 4) * 8;
    // B (16 tokens x 16 dims as [token][dim]): matrices (tokens 0-7, dims 0-7), (0-7, 8-15), (8-15, 0-7), (8-15, 8-15)
    const __half *bp = cs + (size_t)(tok0 + (lane & 7) + ((lane >> 4) << 3)) * cp + ((lane >> 3) & 1) * 8;
    for (int k0 = 0; k0 < DK; k0 += 16) {
      uint32_t ah[4], al[4], bb[4];
      ldsm_x4(ah, a_hi + k0);
      ldsm_x4(al, a_lo + k0);
      ldsm_x4(bb, bp + k0);
      mma16816(c0, ah, bb[0], bb[1]);
      mma16816(c0, al, bb[0], bb[1]);
      mma16816(c1, ah, bb[2], bb[3]);
      mma16816(c1, al, bb[2], bb[3]);
    }
    // accumulator layout: rows lane / 4 and lane / 4 + 8, columns 2 (lane % 4), + 1 of each n8 tile
    const int r0 = lane >> 2, cc = 2 * (lane & 3);
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int ta = tok0 + cc + j, tb = tok0 + 8 + cc + j;
      sc[r0 * MLA_SPLIT + ta] = ta < n ? c0[j] * scale : -CUDART_INF_F;
      sc[(r0 + 8) * MLA_SPLIT + ta] = ta < n ? c0[2 + j] * scale : -CUDART_INF_F;
      sc[r0 * MLA_SPLIT + tb] = tb < n ? c1[j] * scale : -CUDART_INF_F;
      sc[(r0 + 8) * MLA_SPLIT + tb] = tb < n ? c1[2 + j] * scale : -CUDART_INF_F;
    }
  }
  __syncthreads();

  // ---- softmax of the split per head (warp w: heads 2 w, 2 w + 1); weights as fp16 hi + lo rows
  for (int h = 2 * warp; h < 2 * warp + 2; ++h) {
    float v[4], m = -CUDART_INF_F;
#pragma unroll
    for (int k = 0; k < 4; ++k) { v[k] = sc[h * MLA_SPLIT + lane + 32 * k]; m = fmaxf(m, v[k]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float p = expf(v[k] - m);
      const __half hi = __float2half_rn(p);
      ph[h * pp + lane + 32 * k] = hi;
      pl[h * pp + lane + 32 * k] = __float2half_rn(p - __half2float(hi));
      l += p;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) { red[h] = m; red[MLA_NH + h] = l; }
  }
  __syncthreads();

  // ---- O[16 heads][dims 64 warp ..] = P[16 x 128 tokens] * C[128 tokens x dims]: eight n8 tiles per warp and pass
  for (int dbase = 64 * warp; dbase < d_c; dbase += 64 * (MLA_THREADS / 32)) {
    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { acc[j][0] = 0.f; acc[j][1] = 0.f; acc[j][2] = 0.f; acc[j][3] = 0.f; }
    const __half *a_hi = ph + (size_t)(lane & 15) * pp + (lane >> 4) * 8;
    const __half *a_lo = pl + (size_t)(lane & 15) * pp + (lane >> 4) * 8;
    // B (16 tokens x 16 dims stored [token][dim], read transposed): matrices (tokens 0-7, dims 0-7), (8-15, 0-7),
    // (0-7, 8-15), (8-15, 8-15)
    const __half *bp = cs + (size_t)((lane & 7) + ((lane >> 3) & 1) * 8) * cp + dbase + (lane >> 4) * 8;
    for (int k0 = 0; k0 < MLA_SPLIT; k0 += 16) {
      uint32_t ah[4], al[4];
      ldsm_x4(ah, a_hi + k0);
      ldsm_x4(al, a_lo + k0);
#pragma unroll
      for (int j = 0; j < 4; ++j) {                  // 16 dims per ldmatrix: two n8 tiles
        uint32_t bb[4];
        ldsm_x4_t(bb, bp + (size_t)k0 * cp + 16 * j);
        mma16816(acc[2 * j], ah, bb[0], bb[1]);
        mma16816(acc[2 * j], al, bb[0], bb[1]);
        mma16816(acc[2 * j + 1], ah, bb[2], bb[3]);
        mma16816(acc[2 * j + 1], al, bb[2], bb[3]);
      }
    }
    const int r0 = lane >> 2, cc = 2 * (lane & 3);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int d = dbase + 8 * j + cc;
      if (r0 < n_heads)
        *reinterpret_cast<float2 *>(part_o + (((size_t)b * max_splits + s) * n_heads + r0) * d_c + d) = make_float2(acc[j][0], acc[j][1]);
      if (r0 + 8 < n_heads)
        *reinterpret_cast<float2 *>(part_o + (((size_t)b * max_splits + s) * n_heads + r0 + 8) * d_c + d) = make_float2(acc[j][2], acc[j][3]);
    }
  }
  if (tid < n_heads) part_ml[((size_t)b * max_splits + s) * n_heads + tid] = make_float2(red[tid], red[MLA_NH + tid]);
}

// ---------------------------------------------------------------- pipelined version of the same path
// One CTA of 16 warps per (row, chunk of MLA_CHUNK cached tokens).  The chunk's tiles of 64 tokens stream through
// two shared-memory buffers with cp.async (tile i + 1 loads while tile i is computed); the softmax runs online
// over the tiles in ascending order (running maximum M, sum l and output O per head, O in the mma accumulators).
// Instruction issue and shared-memory traffic are the scarce resources (every operand of mma.sync passes through
// ldmatrix), so the queries pass through shared memory once per chunk only: warp w keeps the fp16 hi / lo A fragments of K group w & 3 (a quarter of the k16 steps
// of d_c + d_r) in registers for the whole chunk and multiplies them with tokens 16 (w >> 2) .. + 15 of each tile;
// the four K groups' partial scores are added in a fixed order by the softmax.  The cache tile is read once for
// the scores and once (transposed) for the output: warp w owns dims 32 w .. 32 w + 31 of O.  The chunk's
// (M, l, O) goes to the workspace; chunks are combined in ascending order.  Chunk and tile sizes are fixed, so a
// row's arithmetic depends on its own context length only.
constexpr int MLA_CHUNK = 512;
constexpr int MLA_TILE = 64;
constexpr int MLA_TP = MLA_TILE + 8;   // halfs per weight row
constexpr int MLA_SP = MLA_TILE + 8;   // floats per partial-score row (conflict-free float2 stores)
constexpr int MLA_KG = 4;              // K groups
constexpr int MLA_CTHREADS = 512;     // 16 warps
constexpr int MLA_KS = 9;              // k16 steps per K group at most: d_c + d_r <= 576

__device__ __forceinline__ void split_half2(float2 v, uint32_t &hi, uint32_t &lo) {
  const __half2 h = __floats2half2_rn(v.x, v.y);
  const float2 back = __half22float2(h);
  const __half2 l = __floats2half2_rn(v.x - back.x, v.y - back.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

// DC, DR: the latent and rotary widths at compile time (strides and shared-memory offsets fold into the
// instructions' immediates), or 0, 0 for widths taken from the arguments.
template <bool PAIRS, int DC, int DR>
__global__ void __launch_bounds__(MLA_CTHREADS, 1)
mla_chunk_mma_kernel(const float *__restrict__ q_lat, const float *__restrict__ q_rope, const __half *__restrict__ cache,
                     const int *__restrict__ ctx, int n_heads, int d_c, int d_r, int max_context, int max_chunks, float scale,
                     float *__restrict__ part_o, float2 *__restrict__ part_ml) {
  const int ch = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_ctx = min(ctx[b], max_context);   // a context beyond the cache is cut, never read
  const int t_begin = ch * MLA_CHUNK;
  if (t_begin >= n_ctx) return;
  const int n_chunk = min(MLA_CHUNK, n_ctx - t_begin);
  const int n_tiles = (n_chunk + MLA_TILE - 1) / MLA_TILE;
  if (DC) { d_c = DC; d_r = DR; }
  const int DK = d_c + d_r, cp = DK + MLA_CP;
  extern __shared__ __align__(16) unsigned char smem[];
  __half *cs = reinterpret_cast<__half *>(smem);                     // [2][64][cp]
  const uint32_t cs_s = (uint32_t)__cvta_generic_to_shared(cs);      // 32-bit shared-space addresses for ldmatrix / cp.async
  __half *ph = cs + (size_t)2 * MLA_TILE * cp;                       // [16][MLA_TP] weights hi, then the same for lo
  float *sc = reinterpret_cast<float *>(ph + (size_t)2 * MLA_NH * MLA_TP);   // [4 K groups][16][MLA_SP] partial scores
  float *run_m = sc + MLA_KG * MLA_NH * MLA_SP;                      // [16] running maxima
  float *run_l = run_m + MLA_NH;                                     // [16] running sums
  float *fac = run_l + MLA_NH;                                       // [16] rescale factors of the current tile
  const uint32_t ph_s = (uint32_t)__cvta_generic_to_shared(ph);
  const int r0 = lane >> 2, cc = 2 * (lane & 3);

  auto load_tile = [&](int ti) {
    const int t0 = t_begin + ti * MLA_TILE;
    const int n = min(MLA_TILE, n_ctx - t0);
    const uint32_t dst_s = cs_s + (uint32_t)((ti & 1) * MLA_TILE * cp * 2) + lane * 16;
    const int vecs = DK / 8;
    const __half *src = cache + ((size_t)b * max_context + t0) * DK + lane * 8;
    // warp w: tokens w, w + 16, ...; its lanes the 16-byte pieces of the row
#pragma unroll
    for (int t = warp; t < MLA_TILE; t += MLA_CTHREADS / 32) {
      const uint32_t d = dst_s + (uint32_t)(t * cp * 2);
      if (t < n) {
        const __half *g = src + (size_t)t * DK;
#pragma unroll 3
        for (int j = lane; j < vecs; j += 32)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d + (uint32_t)(j - lane) * 16), "l"(g + (j - lane) * 8) : "memory");
      } else {
#pragma unroll 3
        for (int j = lane; j < vecs; j += 32)
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(d + (uint32_t)(j - lane) * 16), "r"(0u) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  load_tile(0);

  // ---- the row's queries, fp32, through the second tile buffer (free until the loop starts): coalesced 16-byte
  // loads, all of a thread's loads in flight at once
  const int qp = DK + 8;                             // floats per staged query row
  float *qs = reinterpret_cast<float *>(cs + (size_t)MLA_TILE * cp);   // [16][qp] <= one tile buffer
  {
    const float *gl = q_lat + (size_t)b * n_heads * d_c, *gr = q_rope + (size_t)b * n_heads * d_r;
    const int quads = MLA_NH * DK / 4;               // a quad lies in one head and wholly in its latent or rotary part
#pragma unroll 5
    for (int i = tid; i < quads; i += MLA_CTHREADS) {
      const int h = (4 * i) / DK, d = 4 * i - h * DK;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (h < n_heads)
        v = d < d_c ? *reinterpret_cast<const float4 *>(gl + (size_t)h * d_c + d)
                    : *reinterpret_cast<const float4 *>(gr + (size_t)h * d_r + (d - d_c));
      *reinterpret_cast<float4 *>(qs + (size_t)h * qp + d) = v;
    }
  }
  __syncthreads();
  // ---- this warp's query fragments (A operand of m16n8k16: rows = heads, k = 16 dims per step), hi and lo
  const int kg = warp & (MLA_KG - 1), tg = warp >> 2;   // tg 0..3: tokens 16 tg .. 16 tg + 15 of a tile
  const int ksteps = DK / 16, per_group = (ksteps + MLA_KG - 1) / MLA_KG;
  const int my_first = kg * per_group, my_steps = max(0, min(per_group, ksteps - my_first));
  uint32_t qa_hi[MLA_KS][4], qa_lo[MLA_KS][4];
#pragma unroll
  for (int i = 0; i < MLA_KS; ++i) {
    float2 v[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    if (i < my_steps) {
      const float *base = qs + (my_first + i) * 16 + cc;
      v[0] = *reinterpret_cast<const float2 *>(base + (size_t)r0 * qp);
      v[1] = *reinterpret_cast<const float2 *>(base + (size_t)(r0 + 8) * qp);
      v[2] = *reinterpret_cast<const float2 *>(base + (size_t)r0 * qp + 8);
      v[3] = *reinterpret_cast<const float2 *>(base + (size_t)(r0 + 8) * qp + 8);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) split_half2(v[j], qa_hi[i][j], qa_lo[i][j]);
  }
  __syncthreads();                                   // the buffer is free for the second tile
  if (tid < MLA_NH) { run_m[tid] = -CUDART_INF_F; run_l[tid] = 0.f; }

  // this warp's output accumulators: dims dbase .. dbase + 31 of all heads (only warps with dbase < d_c have any)
  const int dbase = 32 * warp;
  float acc[4][4];
#pragma unroll
  for (int j = 0; j < 4; ++j) { acc[j][0] = 0.f; acc[j][1] = 0.f; acc[j][2] = 0.f; acc[j][3] = 0.f; }

  for (int ti = 0; ti < n_tiles; ++ti) {
    if (ti + 1 < n_tiles) {
      load_tile(ti + 1);                             // into the other buffer: its readers passed the loop's last barrier
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                 // tile ti is in shared memory
    const uint32_t ct_s = cs_s + (uint32_t)((ti & 1) * MLA_TILE * cp * 2);
    const int n = min(MLA_TILE, n_chunk - ti * MLA_TILE);
    // ---- partial scores of K group kg for heads x tokens 16 tg .. 16 tg + 15 (two n8 tiles, hi and lo chains)
    {
      float c_hi[2][4], c_lo[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) { c_hi[j][e] = 0.f; c_lo[j][e] = 0.f; }
      // B (16 tokens x 16 dims as [token][dim]): matrices (tokens 0-7, dims 0-7), (0-7, 8-15), (8-15, 0-7), (8-15, 8-15)
      const uint32_t bp = ct_s + 2u * (uint32_t)((16 * tg + (lane & 7) + ((lane >> 4) << 3)) * cp + ((lane >> 3) & 1) * 8 + my_first * 16);
#pragma unroll
      for (int i = 0; i < MLA_KS; ++i) {
        if (i < my_steps) {
          uint32_t b0[4];
          ldsm_x4(b0, bp + i * 32);
          mma16816(c_hi[0], qa_hi[i], b0[0], b0[1]);
          mma16816(c_hi[1], qa_hi[i], b0[2], b0[3]);
          if (PAIRS) {
            mma16816(c_lo[0], qa_lo[i], b0[0], b0[1]);
            mma16816(c_lo[1], qa_lo[i], b0[2], b0[3]);
          }
        }
      }
      float *so = sc + (size_t)kg * MLA_NH * MLA_SP;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int t = 16 * tg + 8 * j + cc;
        *reinterpret_cast<float2 *>(so + r0 * MLA_SP + t) = make_float2(c_hi[j][0] + c_lo[j][0], c_hi[j][1] + c_lo[j][1]);
        *reinterpret_cast<float2 *>(so + (r0 + 8) * MLA_SP + t) = make_float2(c_hi[j][2] + c_lo[j][2], c_hi[j][3] + c_lo[j][3]);
      }
    }
    __syncthreads();
    // ---- online softmax: warp w = head w; the K groups' parts are added in a fixed order
    {
      const int h = warp;
      const float *s0 = sc + h * MLA_SP, *s1 = s0 + MLA_NH * MLA_SP, *s2 = s1 + MLA_NH * MLA_SP, *s3 = s2 + MLA_NH * MLA_SP;
      const float v0 = lane < n ? ((s0[lane] + s1[lane]) + (s2[lane] + s3[lane])) * scale : -CUDART_INF_F;
      const float v1 = lane + 32 < n ? ((s0[lane + 32] + s1[lane + 32]) + (s2[lane + 32] + s3[lane + 32])) * scale : -CUDART_INF_F;
      float m = fmaxf(v0, v1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      const float M_old = run_m[h], M_new = fmaxf(M_old, m);
      const float p0 = __expf(v0 - M_new), p1 = __expf(v1 - M_new);
      const __half h0 = __float2half_rn(p0), h1 = __float2half_rn(p1);
      __half *wh = ph + (size_t)h * MLA_TP, *wl = ph + (size_t)(MLA_NH + h) * MLA_TP;
      wh[lane] = h0;
      wh[lane + 32] = h1;
      if (PAIRS) {
        wl[lane] = __float2half_rn(p0 - __half2float(h0));
        wl[lane + 32] = __float2half_rn(p1 - __half2float(h1));
      }
      // without the lo parts the sum runs over the rounded weights, so that numerator and denominator agree
      float l = PAIRS ? p0 + p1 : __half2float(h0) + __half2float(h1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
      __syncwarp();
      if (lane == 0) {
        const float f = __expf(M_old - M_new);       // 0 the first time (M_old = -inf)
        fac[h] = f;
        run_l[h] = run_l[h] * f + l;
        run_m[h] = M_new;
      }
    }
    __syncthreads();
    // ---- O = O * f + P[16 x 64 tokens] * C[64 tokens x dims]
    if (dbase < d_c) {
      const float f0 = fac[r0], f1 = fac[r0 + 8];
#pragma unroll
      for (int j = 0; j < 4; ++j) { acc[j][0] *= f0; acc[j][1] *= f0; acc[j][2] *= f1; acc[j][3] *= f1; }
      const uint32_t a_hi = ph_s + 2u * (uint32_t)((lane & 15) * MLA_TP + (lane >> 4) * 8);
      const uint32_t a_lo = a_hi + 2u * MLA_NH * MLA_TP;
      // B (16 tokens x 16 dims stored [token][dim], read transposed): matrices (tokens 0-7, dims 0-7), (8-15, 0-7),
      // (0-7, 8-15), (8-15, 8-15)
      const uint32_t bp = ct_s + 2u * (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * cp + dbase + (lane >> 4) * 8);
#pragma unroll
      for (int k0 = 0; k0 < MLA_TILE; k0 += 16) {
        uint32_t ah[4], al[4];
        ldsm_x4(ah, a_hi + 2 * k0);
        if (PAIRS) ldsm_x4(al, a_lo + 2 * k0);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          uint32_t bb[4];
          ldsm_x4_t(bb, bp + 2u * (uint32_t)(k0 * cp + 16 * j));
          mma16816(acc[2 * j], ah, bb[0], bb[1]);
          mma16816(acc[2 * j + 1], ah, bb[2], bb[3]);
          if (PAIRS) {
            mma16816(acc[2 * j], al, bb[0], bb[1]);
            mma16816(acc[2 * j + 1], al, bb[2], bb[3]);
          }
        }
      }
    }
    // the next iteration starts a load into the other buffer and rewrites the score and weight tiles: everyone
    // must have finished this iteration's reads of the weights (and the previous one's of that buffer) first
    __syncthreads();
  }
  if (dbase < d_c) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int d = dbase + 8 * j + cc;
      if (r0 < n_heads)
        *reinterpret_cast<float2 *>(part_o + (((size_t)b * max_chunks + ch) * n_heads + r0) * d_c + d) = make_float2(acc[j][0], acc[j][1]);
      if (r0 + 8 < n_heads)
        *reinterpret_cast<float2 *>(part_o + (((size_t)b * max_chunks + ch) * n_heads + r0 + 8) * d_c + d) = make_float2(acc[j][2], acc[j][3]);
    }
  }
  if (tid < n_heads) part_ml[((size_t)b * max_chunks + ch) * n_heads + tid] = make_float2(run_m[tid], run_l[tid]);
}

size_t mla_chunk_smem_bytes(int d_c, int d_r) {
  const int DK = d_c + d_r;
  return (size_t)2 * MLA_TILE * (DK + MLA_CP) * 2 + (size_t)2 * MLA_NH * MLA_TP * 2 +
         (size_t)MLA_KG * MLA_NH * MLA_SP * 4 + 3 * MLA_NH * 4 + 64;   // + slack: the last row's ldmatrix may read past its padding
}

size_t mla_mma_smem_bytes(int d_c, int d_r) {
  const int DK = d_c + d_r;
  return (size_t)(MLA_SPLIT + 2 * MLA_NH) * (DK + MLA_CP) * 2 + (size_t)2 * MLA_NH * (MLA_SPLIT + MLA_PP) * 2 +
         (size_t)MLA_NH * MLA_SPLIT * 4 + 2 * MLA_NH * 4;
}

// One CTA per (head, row): the row's splits in ascending order.
__global__ void __launch_bounds__(MLA_THREADS)
mla_combine_kernel(const float *__restrict__ part_o, const float2 *__restrict__ part_ml, const int *__restrict__ ctx,
                   int n_heads, int d_c, int max_splits, int split_len, float *__restrict__ o_lat) {
  const int h = blockIdx.x, b = blockIdx.y;
  const int n_ctx = ctx[b];
  if (n_ctx <= 0) return;
  const int ns = min((n_ctx + split_len - 1) / split_len, max_splits);   // as the piece kernels cut it
  const float2 *ml = part_ml + (size_t)b * max_splits * n_heads + h;
  const float *po = part_o + ((size_t)b * max_splits * n_heads + h) * d_c;
  const size_t o_stride = (size_t)n_heads * d_c;     // floats between a head's consecutive pieces
  constexpr int FAST = 16;                           // pieces whose weights fit in registers
  if (ns <= FAST) {
    // all (max, sum) pairs in one round trip, the weights once, then all pieces of a dim in one round trip;
    // the arithmetic (maximum first, ascending sums) is that of the general loop below
    float2 v[FAST];
#pragma unroll
    for (int s = 0; s < FAST; ++s) v[s] = s < ns ? ml[(size_t)s * n_heads] : make_float2(-CUDART_INF_F, 0.f);
    float M = -CUDART_INF_F;
#pragma unroll
    for (int s = 0; s < FAST; ++s) M = fmaxf(M, v[s].x);
    float w[FAST], den = 0.f;
#pragma unroll
    for (int s = 0; s < FAST; ++s) {
      w[s] = s < ns ? expf(v[s].x - M) : 0.f;
      if (s < ns) den += w[s] * v[s].y;
    }
    const float inv = 1.f / den;
    for (int d = 4 * threadIdx.x; d < d_c; d += 4 * blockDim.x) {
      float4 x[FAST];
#pragma unroll
      for (int s = 0; s < FAST; ++s)
        x[s] = s < ns ? *reinterpret_cast<const float4 *>(po + (size_t)s * o_stride + d) : make_float4(0.f, 0.f, 0.f, 0.f);
      float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < FAST; ++s) {
        if (s < ns) { o.x = fmaf(w[s], x[s].x, o.x); o.y = fmaf(w[s], x[s].y, o.y); o.z = fmaf(w[s], x[s].z, o.z); o.w = fmaf(w[s], x[s].w, o.w); }
      }
      *reinterpret_cast<float4 *>(o_lat + ((size_t)b * n_heads + h) * d_c + d) = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
    }
    return;
  }
  float M = -CUDART_INF_F;
  for (int s = 0; s < ns; ++s) M = fmaxf(M, ml[(size_t)s * n_heads].x);
  float den = 0.f;
  for (int s = 0; s < ns; ++s) den += expf(ml[(size_t)s * n_heads].x - M) * ml[(size_t)s * n_heads].y;
  const float inv = 1.f / den;
  for (int d = threadIdx.x; d < d_c; d += blockDim.x) {
    float o = 0.f;
    for (int s = 0; s < ns; ++s) o = fmaf(expf(ml[(size_t)s * n_heads].x - M), po[(size_t)s * o_stride + d], o);
    o_lat[((size_t)b * n_heads + h) * d_c + d] = o * inv;
  }
}

size_t mla_smem_bytes(int d_c, int d_r) {
  const int DK = d_c + d_r;
  return (size_t)DK * MLA_NH * 4 + (size_t)MLA_SPLIT * MLA_NH * 4 + 2 * MLA_NH * 4 + (size_t)MLA_SPLIT * (DK + 2) * 2;
}

}  // namespace

extern "C" {

int64_t corun_mla_workspace_floats(int32_t B, int32_t n_heads, int32_t d_latent, int32_t max_context) {
  if (B < 1 || n_heads < 1 || d_latent < 1 || max_context < 1) return 0;
  const int64_t splits = (max_context + MLA_SPLIT - 1) / MLA_SPLIT;
  return (int64_t)B * splits * n_heads * (d_latent + 2);
}

int corun_mla_attend(const float *q_lat, const float *q_rope, const void *cache, const int32_t *ctx, int32_t B,
                     int32_t n_heads, int32_t d_latent, int32_t d_rope, int32_t max_context, float scale, float *o_lat,
                     float *ws, int32_t operand_pairs, void *cuda_stream) {
  if (!q_lat || !q_rope || !cache || !ctx || !o_lat || !ws || B < 1 || B > 65535 || n_heads < 4 || n_heads > MLA_NH ||
      n_heads % 4 || d_latent < 64 || d_latent > 512 || d_latent % 64 || d_rope < 8 || d_rope > 64 || d_rope % 8 ||
      max_context < 1 || (operand_pairs != 0 && operand_pairs != 1))
    return CORUN_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int max_splits = (max_context + MLA_SPLIT - 1) / MLA_SPLIT;
  // the warp-level tensor path needs whole k16 steps and 64-dim passes; otherwise (or on request) plain FMAs
  if (reinterpret_cast<uintptr_t>(cache) % 16 || reinterpret_cast<uintptr_t>(q_lat) % 16 || reinterpret_cast<uintptr_t>(q_rope) % 16 ||
      reinterpret_cast<uintptr_t>(o_lat) % 16 || reinterpret_cast<uintptr_t>(ws) % 16)
    return CORUN_EINVAL;
  auto env_on = [](const char *name) { const char *v = getenv(name); return v && atoi(v) != 0; };
  // single fp16 operands exist on the pipelined tensor path only
  if (!operand_pairs && (d_rope % 16 != 0 || env_on("CORUN_MLA_FMA") || env_on("CORUN_MLA_UNPIPELINED"))) return CORUN_EINVAL;
  const bool use_mma = d_rope % 16 == 0 && !env_on("CORUN_MLA_FMA");
  const bool use_chunk = use_mma && !env_on("CORUN_MLA_UNPIPELINED");
  float *part_o = ws;
  if (use_chunk) {
    // pipelined path: chunks of MLA_CHUNK tokens (the workspace, sized for 128-token splits, is large enough)
    const int max_chunks = (max_context + MLA_CHUNK - 1) / MLA_CHUNK;
    const size_t smem = mla_chunk_smem_bytes(d_latent, d_rope);
    // the DeepSeek-V2 / V3 widths are compiled in; any other shape takes the kernel with run-time widths
    const bool v2 = d_latent == 512 && d_rope == 64;
    auto kern = v2 ? (operand_pairs ? mla_chunk_mma_kernel<true, 512, 64> : mla_chunk_mma_kernel<false, 512, 64>)
                   : (operand_pairs ? mla_chunk_mma_kernel<true, 0, 0> : mla_chunk_mma_kernel<false, 0, 0>);
    cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ce != cudaSuccess) { corun::g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
    float2 *part_ml = reinterpret_cast<float2 *>(ws + (size_t)B * max_chunks * n_heads * d_latent);
    kern<<<dim3(max_chunks, B), MLA_CTHREADS, smem, st>>>(q_lat, q_rope, (const __half *)cache, ctx, n_heads, d_latent, d_rope,
                                                        max_context, max_chunks, scale, part_o, part_ml);
    mla_combine_kernel<<<dim3(n_heads, B), 128, 0, st>>>(part_o, part_ml, ctx, n_heads, d_latent, max_chunks, MLA_CHUNK,
                                                                o_lat);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) { corun::g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
    return CORUN_OK;
  }
  const size_t smem = use_mma ? mla_mma_smem_bytes(d_latent, d_rope) : mla_smem_bytes(d_latent, d_rope);
  cudaError_t ce = use_mma ? cudaFuncSetAttribute(mla_split_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                           : cudaFuncSetAttribute(mla_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (ce != cudaSuccess) { corun::g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  float2 *part_ml = reinterpret_cast<float2 *>(ws + (size_t)B * max_splits * n_heads * d_latent);
  if (use_mma)
    mla_split_mma_kernel<<<dim3(max_splits, B), MLA_THREADS, smem, st>>>(q_lat, q_rope, (const __half *)cache, ctx, n_heads,
                                                                        d_latent, d_rope, max_context, max_splits, scale, part_o,
                                                                        part_ml);
  else
    mla_split_kernel<<<dim3(max_splits, B), MLA_THREADS, smem, st>>>(q_lat, q_rope, (const __half *)cache, ctx, n_heads, d_latent,
                                                                    d_rope, max_context, max_splits, scale, part_o, part_ml);
  mla_combine_kernel<<<dim3(n_heads, B), 128, 0, st>>>(part_o, part_ml, ctx, n_heads, d_latent, max_splits, MLA_SPLIT,
                                                              o_lat);
  ce = cudaGetLastError();
  if (ce != cudaSuccess) { corun::g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return CORUN_OK;
}

}  // extern "C"
