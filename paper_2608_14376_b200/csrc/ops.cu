// Non-GEMM kernels of the row program: residual + RMSNorm, RoPE + KV append,
// request-local split-KV paged attention with a fixed-order combine, SwiGLU,
// seeded sampling, decode bookkeeping.  Every reduction has one fixed order
// that depends on the row's own data and the model shape only; no float atomics.
#include "ops.cuh"

#include "checks.cuh"
#include "launch.cuh"
#include "ptx.cuh"

#include <cooperative_groups.h>

#include <cstdlib>
#include <math_constants.h>

namespace corun {

namespace {

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// ---------------------------------------------------------------- residual + RMSNorm
constexpr int NORM_MAX_THREADS = 1024;

__device__ __forceinline__ void store_split4(float4 y, __nv_bfloat16 *hi, __nv_bfloat16 *lo) {
  __nv_bfloat16 a[4], b[4];
  split_bf16(y.x, a[0], b[0]);
  split_bf16(y.y, a[1], b[1]);
  split_bf16(y.z, a[2], b[2]);
  split_bf16(y.w, a[3], b[3]);
  *reinterpret_cast<uint2 *>(hi) = *reinterpret_cast<const uint2 *>(a);
  *reinterpret_cast<uint2 *>(lo) = *reinterpret_cast<const uint2 *>(b);
}

// One CTA per row, one float4 per thread and pass (H % 4 == 0).  Sum of squares: thread-serial over
// the thread's elements (ascending), xor-butterfly in the warp, warp totals in ascending order.
__global__ void __launch_bounds__(NORM_MAX_THREADS)
resid_norm_kernel(float *__restrict__ h, int H, const __nv_bfloat16 *__restrict__ embed, Rows rows, GemmOut prev,
                  int first, const __nv_bfloat16 *__restrict__ gains, float eps, __nv_bfloat16 *__restrict__ out_hi,
                  __nv_bfloat16 *__restrict__ out_lo) {
  griddep_launch_dependents();
  griddep_wait();
  __shared__ float scratch[NORM_MAX_THREADS / 32];
  const int r = blockIdx.x;
  float *hr = h + (size_t)r * H;
  float ss = 0.f;
  if (first) {
    const __nv_bfloat16 *e = embed + (size_t)rows.token[r] * H;
    for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
      const uint2 raw = *reinterpret_cast<const uint2 *>(e + i);
      const __nv_bfloat162 *b2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
      const float2 lo2 = __bfloat1622float2(b2[0]), hi2 = __bfloat1622float2(b2[1]);
      const float4 x = make_float4(lo2.x, lo2.y, hi2.x, hi2.y);
      *reinterpret_cast<float4 *>(hr + i) = x;
      ss = fmaf(x.x, x.x, ss); ss = fmaf(x.y, x.y, ss); ss = fmaf(x.z, x.z, ss); ss = fmaf(x.w, x.w, ss);
    }
  } else {
    for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
      const float4 d = gemm_load4(prev, r, i);
      float4 x = *reinterpret_cast<const float4 *>(hr + i);
      x.x += d.x; x.y += d.y; x.z += d.z; x.w += d.w;
      *reinterpret_cast<float4 *>(hr + i) = x;
      ss = fmaf(x.x, x.x, ss); ss = fmaf(x.y, x.y, ss); ss = fmaf(x.z, x.z, ss); ss = fmaf(x.w, x.w, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  if (lane == 0) scratch[warp] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < nwarps; ++w) tot += scratch[w];
  const float inv = rsqrtf(tot / (float)H + eps);
  for (int i = threadIdx.x * 4; i < H; i += blockDim.x * 4) {
    const float4 x = *reinterpret_cast<const float4 *>(hr + i);   // written by this same thread above
    const uint2 raw = *reinterpret_cast<const uint2 *>(gains + i);
    const __nv_bfloat162 *g2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    const float2 ga = __bfloat1622float2(g2[0]), gb = __bfloat1622float2(g2[1]);
    const float4 y = make_float4(x.x * inv * ga.x, x.y * inv * ga.y, x.z * inv * gb.x, x.w * inv * gb.y);
    store_split4(y, out_hi + (size_t)r * H + i, out_lo + (size_t)r * H + i);
  }
}

// ---------------------------------------------------------------- RoPE + KV append
// One CTA per (head, row): heads 0..nq-1 are q, nq..nq+nkv-1 are k, the rest are v; hd/2 threads.
__global__ void __launch_bounds__(64)
qkv_post_kernel(GemmOut qkv, Rows rows, const float2 *__restrict__ rope_tab, int nq, KvLayout kv, int layer,
                float *__restrict__ q_out, int *status) {
  griddep_launch_dependents();
  griddep_wait();
  const int head = blockIdx.x, r = blockIdx.y, i = threadIdx.x;
  const int hd = kv.hd, half = hd >> 1, nkv = kv.n_kv;
  const int pos = rows.pos[r];
  const bool active = rows.active[r] != 0;
  if (head >= nq && !active) return;               // padding rows write no cache
  const int col = head * hd + i;                   // q, k and v heads are contiguous in the GEMM output
  const float a = gemm_load(qkv, r, col), b = gemm_load(qkv, r, col + half);
  if (head < nq) {
    const float2 t = rope_tab[(size_t)pos * half + i];   // (cos, sin)
    float *q = q_out + (size_t)r * nq * hd + col;
    q[0] = a * t.x - b * t.y;
    q[half] = a * t.y + b * t.x;
    return;
  }
#ifdef CORUN_CHECKED
  if (!check_slot_pos(rows.slot[r], kv.n_slots, pos, kv.max_blocks, KV_BLOCK)) {   // the write is skipped
    atomicCAS(status, 0, DEV_BAD_INDEX);
    return;
  }
#endif
  const int blk = kv.block_table[(size_t)rows.slot[r] * kv.max_blocks + pos / KV_BLOCK];
#ifdef CORUN_CHECKED
  if (!check_page(blk, kv.pool_blocks)) {
    atomicCAS(status, 0, DEV_BAD_INDEX);
    return;
  }
#endif
  __half *page = kv.pool + (size_t)layer * kv.layer_stride + (size_t)blk * 2 * nkv * KV_BLOCK * hd;
  const int tok = pos % KV_BLOCK;
  if (head < nq + nkv) {
    const float2 t = rope_tab[(size_t)pos * half + i];
    const int g = head - nq;
    page[kv_k_off(hd, g, tok, i)] = __float2half_rn(a * t.x - b * t.y);
    page[kv_k_off(hd, g, tok, i + half)] = __float2half_rn(a * t.y + b * t.x);
  } else {
    const int g = head - nq - nkv;
    page[kv_v_off(nkv, hd, g, tok, i)] = __float2half_rn(a);
    page[kv_v_off(nkv, hd, g, tok, i + half)] = __float2half_rn(b);
  }
}

// ---------------------------------------------------------------- SwiGLU
__global__ void __launch_bounds__(256)
swiglu_kernel(GemmOut gu, int F, __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int r = blockIdx.y;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= F) return;
  const float4 g = gemm_load4(gu, r, i), u = gemm_load4(gu, r, F + i);
  const float4 y = make_float4(g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                               g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w);
  store_split4(y, out_hi + (size_t)r * F + i, out_lo + (size_t)r * F + i);
}

__global__ void split_kernel(const float *__restrict__ x, size_t n, __nv_bfloat16 *__restrict__ hi,
                             __nv_bfloat16 *__restrict__ lo) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  __nv_bfloat16 a, b;
  split_bf16(x[i], a, b);
  hi[i] = a;
  lo[i] = b;
}

// ---------------------------------------------------------------- R(seed, t) and S
// Philox4x32-10 (Salmon et al., SC'11): multipliers 0xD2511F53 / 0xCD9E8D57,
// key increments 0x9E3779B9 / 0xBB67AE85.  The variate is the top 24 bits of word 0.
__device__ __forceinline__ uint32_t philox_u24(uint64_t seed, uint64_t t) {
  uint32_t c0 = (uint32_t)t, c1 = (uint32_t)(t >> 32), c2 = 0u, c3 = 0u;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0 >> 8;
}

__global__ void variate_kernel(uint64_t seed, uint64_t t, uint32_t *out) { *out = philox_u24(seed, t); }

constexpr int SMP_THREADS = 1024;
constexpr int SMP_BINS = 2048;

// order-preserving map float -> uint32 (larger float = larger key)
__device__ __forceinline__ uint32_t ordered_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum over the block (thread order); integer, hence exact.
__device__ __forceinline__ unsigned long long block_excl_scan_u64(unsigned long long v, unsigned long long *wtot /*[32]*/,
                                                                  unsigned long long *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();
  if (lane == 31) wtot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = wtot[lane];
    unsigned long long winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    wtot[lane] = winc - w;   // exclusive warp offsets
    if (lane == 31 && total) *total = winc;
  }
  __syncthreads();
  return wtot[warp] + inc - v;
}

constexpr int SMP_CAND = 2048;   // tokens of the selected coarse bin that are kept in shared memory

struct SmpShared {
  unsigned long long hist[SMP_BINS];
  unsigned int cnt[SMP_BINS];
  unsigned long long wtot[32];
  unsigned long long total, carried, sel_sum;
  float red_val[32];
  int red_idx[32];
  unsigned int kmin, kmax, sel_cnt, n_cand;
  int sel_bin, sel_warp, tie_max_id;
  float cand_x[SMP_CAND];
  int cand_id[SMP_CAND];
  // per-CTA results that the other CTAs of the row's cluster read
  float loc_val; int loc_idx;                     // slice maximum and its lowest id
  unsigned long long loc_total;                   // slice sum of weights
  unsigned long long loc_wtot[32];                // per-warp nucleus weight of the slice, in id order
  // decisions of the cluster's first CTA, read by the others
  int bc_bin, bc_overflow, bc_tie_max_id, bc_sel_rank, bc_sel_warp;
  unsigned int bc_kstar;
  unsigned long long bc_wstar, bc_rdraw, bc_before;
};

// Integer weight of a token: floor(2^40 * exp2(x)), x = fl32(fl32(l - max) * inv_t_log2e).
// exp2 is spelled out so that the integer is the same on every IEEE-754 machine:
// x = n + f with n = rint(x); degree-7 Taylor polynomial of 2^f (ln(2)^k / k! in fp32),
// Horner form, separately rounded multiplies and adds; exact scaling by 2^(n+40).
__device__ __forceinline__ unsigned long long smp_weight(float l, float mx, float inv_t_log2e) {
  const float x = __fmul_rn(__fsub_rn(l, mx), inv_t_log2e);
  if (!(x > -41.5f)) return 0ull;                    // rint(x) <= -42 (ties to even): the weight below is 0 (also NaN)
  const float n = rintf(x);
  const float f = __fsub_rn(x, n);
  float p = 0x1.ffcbfcp-17f;
  p = __fadd_rn(__fmul_rn(p, f), 0x1.430912p-13f);
  p = __fadd_rn(__fmul_rn(p, f), 0x1.5d87fep-10f);
  p = __fadd_rn(__fmul_rn(p, f), 0x1.3b2ab6p-7f);
  p = __fadd_rn(__fmul_rn(p, f), 0x1.c6b08ep-5f);
  p = __fadd_rn(__fmul_rn(p, f), 0x1.ebfbe0p-3f);
  p = __fadd_rn(__fmul_rn(p, f), 0x1.62e430p-1f);
  p = __fadd_rn(__fmul_rn(p, f), 1.0f);
  const int ni = (int)n;
  if (ni < -41) return 0ull;
  const float scale = __int_as_float((ni + 40 + 127) << 23);   // 2^(n+40), exact
  return (unsigned long long)__fmul_rn(p, scale);              // truncation = floor
}

// hist[bin] += w with two 32-bit shared-memory atomics instead of one 64-bit one: the low words wrap modulo 2^32
// and exactly the additions that wrap carry one into the high word, so the 64-bit total is exact whatever the
// order (weights below 2^32 that do not wrap take a single atomic).
__device__ __forceinline__ void smp_hist_add(unsigned long long *h, unsigned long long w) {
  unsigned int *p = reinterpret_cast<unsigned int *>(h);   // p[0]: low word, p[1]: high word
  const unsigned int lo = (unsigned int)w, hi = (unsigned int)(w >> 32);
  const unsigned int old = atomicAdd(p, lo);
  const unsigned int up = hi + ((old + lo < old) ? 1u : 0u);
  if (up) atomicAdd(p + 1, up);
}

// After a histogram pass: finds the first bin (ascending index = descending
// logit) that is non-empty and whose running weight reaches the cut; adds the
// weight of the bins before it to `carried`.  With use_cnt = false a bin counts
// as non-empty when its weight is positive (the coarse pass keeps no counts:
// there the selected bin always has positive weight, because bin 0 holds the
// maximum, whose weight is 2^40).
__device__ void smp_select_bin(SmpShared &sh, unsigned long long cut, bool use_cnt) {
  const int tid = threadIdx.x;
  const unsigned long long a = sh.hist[2 * tid], b = sh.hist[2 * tid + 1];
  unsigned long long tot;
  const unsigned long long before = block_excl_scan_u64(a + b, sh.wtot, &tot);
  if (tid == 0) sh.sel_bin = SMP_BINS;
  __syncthreads();
  const unsigned long long base = sh.carried + before;
  const bool ne0 = use_cnt ? sh.cnt[2 * tid] != 0u : a != 0ull;
  const bool ne1 = use_cnt ? sh.cnt[2 * tid + 1] != 0u : b != 0ull;
  if (ne0 && base + a >= cut) atomicMin(&sh.sel_bin, 2 * tid);
  else if (ne1 && base + a + b >= cut) atomicMin(&sh.sel_bin, 2 * tid + 1);
  __syncthreads();
  const int sel = sh.sel_bin;   // < SMP_BINS: total weight always reaches the cut
  if (sel < SMP_BINS && (sel >> 1) == tid) {
    sh.carried = base + ((sel & 1) ? a : 0ull);
    sh.sel_sum = (sel & 1) ? b : a;
    sh.sel_cnt = use_cnt ? sh.cnt[sel] : 0u;
  }
  __syncthreads();
}

// One refinement step in key space: bins the keys of [kmin, kmax] into SMP_BINS
// equal ranges (descending key = ascending bin), selects the bin where the
// running weight reaches the cut and narrows [kmin, kmax] to it.
struct KeyRange { uint32_t kmin, kmax; };
__device__ __forceinline__ int smp_key_bin(uint32_t k, uint32_t kmin, unsigned long long width) {
  return SMP_BINS - 1 - (int)(((unsigned long long)(k - kmin) * SMP_BINS) / width);
}
__device__ __forceinline__ KeyRange smp_narrow(const SmpShared &sh, uint32_t kmin, unsigned long long width) {
  const unsigned long long j = (unsigned long long)(SMP_BINS - 1 - sh.sel_bin);
  // keys k with floor((k - kmin) * BINS / width) == j
  const unsigned long long lo = (j * width + SMP_BINS - 1) / SMP_BINS;
  const unsigned long long hi = ((j + 1) * width + SMP_BINS - 1) / SMP_BINS - 1;
  return KeyRange{kmin + (uint32_t)lo, kmin + (uint32_t)hi};
}

// Every logit of this CTA's slice of the row, by float4 where the row allows it (V % 4 == 0), else one
// by one.  Units are float4 groups or single ids; the slice is [u_lo, u_hi).
#define SMP_FOREACH(BODY)                                                                  \
  if (vec) {                                                                               \
    _Pragma("unroll 2") for (int i4 = u_lo + tid; i4 < u_hi; i4 += SMP_THREADS) {          \
      const float4 q4 = reinterpret_cast<const float4 *>(lg)[i4];                          \
      const float xs4[4] = {q4.x, q4.y, q4.z, q4.w};                                       \
      _Pragma("unroll") for (int j4 = 0; j4 < 4; ++j4) {                                   \
        const int i = 4 * i4 + j4;                                                         \
        const float x = xs4[j4];                                                           \
        BODY                                                                               \
      }                                                                                    \
    }                                                                                      \
  } else {                                                                                 \
    for (int i = u_lo + tid; i < u_hi; i += SMP_THREADS) {                                 \
      const float x = lg[i];                                                               \
      BODY                                                                                 \
    }                                                                                      \
  }

// Slow tail, used when the selected coarse bin holds more tokens than the
// candidate list (rows with very many equal or nearly equal logits): the
// refinement and the final walk read the whole row every time.
__device__ __noinline__ void smp_tail_full_row(SmpShared &sh, const SampleArgs &a, int r, const float *lg, float mx,
                                               float inv_t_log2e, float scale_a, int bin_a, unsigned long long cut,
                                               uint32_t u24) {
  const int tid = threadIdx.x, V = a.V;
  if (tid == 0) { sh.kmin = 0xffffffffu; sh.kmax = 0u; }
  __syncthreads();
  for (int i = tid; i < V; i += SMP_THREADS) {
    const float x = lg[i];
    if (min(SMP_BINS - 1, (int)((mx - x) * scale_a)) == bin_a) {
      const uint32_t k = ordered_key(x);
      atomicMin(&sh.kmin, k);
      atomicMax(&sh.kmax, k);
    }
  }
  __syncthreads();
  uint32_t kmin = sh.kmin, kmax = sh.kmax;
  for (int pass = 0; pass < 4 && kmax > kmin; ++pass) {
    const unsigned long long width = (unsigned long long)(kmax - kmin) + 1ull;
    __syncthreads();
    for (int i = tid; i < SMP_BINS; i += SMP_THREADS) { sh.hist[i] = 0ull; sh.cnt[i] = 0u; }
    __syncthreads();
    for (int i = tid; i < V; i += SMP_THREADS) {
      const float x = lg[i];
      const uint32_t k = ordered_key(x);
      if (k >= kmin && k <= kmax) {
        const int bin = smp_key_bin(k, kmin, width);
        atomicAdd(&sh.hist[bin], smp_weight(x, mx, inv_t_log2e));
        atomicAdd(&sh.cnt[bin], 1u);
      }
    }
    __syncthreads();
    smp_select_bin(sh, cut, true);
    const KeyRange kr = smp_narrow(sh, kmin, width);
    kmin = kr.kmin; kmax = kr.kmax;
  }
  // Now every token with key == kmin (== kmax) is tied at the nucleus edge.
  const uint32_t kstar = kmin;
  const unsigned long long carried = sh.carried;     // weight of tokens with key > kstar
  const unsigned long long wstar = sh.sel_cnt ? sh.sel_sum / sh.sel_cnt : 0ull;
  unsigned long long m_ties = 1ull;
  if (wstar > 0ull && cut > carried) m_ties = (cut - carried + wstar - 1ull) / wstar;
  if (m_ties < 1ull) m_ties = 1ull;
  if (m_ties > sh.sel_cnt) m_ties = sh.sel_cnt;
  const unsigned long long Z = carried + m_ties * wstar;
  const unsigned long long rdraw = __umul64hi(Z, (unsigned long long)u24 << 40);   // floor(u24 * Z / 2^24)

  // inverse CDF over nucleus members in ascending id order; thread = contiguous id range
  const int per = (V + SMP_THREADS - 1) / SMP_THREADS;
  const int i0 = min(V, tid * per), i1 = min(V, i0 + per);
  unsigned long long nt = 0ull;
  for (int i = i0; i < i1; ++i) nt += (ordered_key(lg[i]) == kstar) ? 1ull : 0ull;
  __syncthreads();
  const unsigned long long ties_before = block_excl_scan_u64(nt, sh.wtot, nullptr);
  unsigned long long ws = 0ull, tr = ties_before;
  for (int i = i0; i < i1; ++i) {
    const float x = lg[i];
    const uint32_t k = ordered_key(x);
    if (k > kstar) ws += smp_weight(x, mx, inv_t_log2e);
    else if (k == kstar) { if (tr < m_ties) ws += wstar; ++tr; }
  }
  __syncthreads();
  const unsigned long long before = block_excl_scan_u64(ws, sh.wtot, nullptr);
  if (rdraw >= before && rdraw < before + ws) {
    unsigned long long run = before;
    tr = ties_before;
    int tok = i1 - 1;
    for (int i = i0; i < i1; ++i) {
      const float x = lg[i];
      const uint32_t k = ordered_key(x);
      unsigned long long w = 0ull;
      if (k > kstar) w = smp_weight(x, mx, inv_t_log2e);
      else if (k == kstar) { if (tr < m_ties) w = wstar; ++tr; }
      run += w;
      if (run > rdraw) { tok = i; break; }
    }
    a.out_token[r] = tok;
  }
}

// Sampling S (top-p nucleus + inverse CDF) of one row per cluster of 1..8 CTAs (a launch attribute), all in integers
// once the weights are formed, so the result does not depend on the order in which threads meet the
// tokens.  Every CTA takes a contiguous slice of the row; the first CTA of the cluster merges what the
// slices found (through distributed shared memory) and takes the decisions.  Four passes over the row:
// maximum; coarse histogram of the weights over (max - logit); collection of the tokens of the bin where
// the running weight reaches the cut (the nucleus edge is then found among those few tokens in shared
// memory); per-warp totals of the nucleus weights in id order, after which one warp walks its range to
// the drawn token.
constexpr int SMP_MAX_CLUSTER = 8;   // the cluster size is a launch attribute (launch_sampler): 2..8 CTAs per row

__global__ void __launch_bounds__(SMP_THREADS, 2) sampler_kernel(SampleArgs a) {
  namespace cg = cooperative_groups;
  griddep_launch_dependents();
  griddep_wait();
  cg::cluster_group cluster = cg::this_cluster();
  const int SMP_CLUSTER = (int)cluster.num_blocks();   // CTAs per row (no value depends on it: integer arithmetic)
  const int r = blockIdx.x / SMP_CLUSTER;
  if (!a.do_sample[r]) return;                     // the same for the whole cluster
  const int rank = (int)cluster.block_rank();
  __shared__ SmpShared sh;
  SmpShared *peer[SMP_MAX_CLUSTER];
#pragma unroll
  for (int k = 0; k < SMP_MAX_CLUSTER; ++k) peer[k] = cluster.map_shared_rank(&sh, k < SMP_CLUSTER ? k : 0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = a.V;
  const float *lg = a.logits + (size_t)r * V;
  const bool vec = (V & 3) == 0 && (((uintptr_t)lg) & 15u) == 0;
  const int units = vec ? (V >> 2) : V;            // float4 groups or single ids
  const int u_lo = (int)(((long long)units * rank) / SMP_CLUSTER), u_hi = (int)(((long long)units * (rank + 1)) / SMP_CLUSTER);

  // ---- argmax, lowest id on ties
  float bv = -CUDART_INF_F;
  int bi = 0x7fffffff;
  SMP_FOREACH(if (x > bv || (x == bv && i < bi)) { bv = x; bi = i; })
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if (lane == 0) { sh.red_val[warp] = bv; sh.red_idx[warp] = bi; }
  __syncthreads();
  if (tid == 0) {
    bv = sh.red_val[0]; bi = sh.red_idx[0];
    for (int w = 1; w < SMP_THREADS / 32; ++w) {
      const float ov = sh.red_val[w];
      const int oi = sh.red_idx[w];
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    sh.loc_val = bv; sh.loc_idx = bi;
  }
  cluster.sync();
  bv = peer[0]->loc_val; bi = peer[0]->loc_idx;
#pragma unroll
  for (int k = 1; k < SMP_MAX_CLUSTER; ++k) {
    if (k >= SMP_CLUSTER) break;
    const float ov = peer[k]->loc_val;
    const int oi = peer[k]->loc_idx;
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  const float temperature = a.temperature[r];
  if (!(temperature > 0.f)) {
    if (rank == 0 && tid == 0) a.out_token[r] = bi;
    cluster.sync();                                // nobody leaves while its shared memory may still be read
    return;
  }
  const float mx = bv;
  const float inv_t_log2e = __fdiv_rn(0x1.715476p+0f, temperature);
  const uint32_t u24 = a.u24_override ? a.u24_override[r] : philox_u24(a.seed[r], (uint64_t)a.step[r]);

  // ---- pass A: bins linear in (max - logit); bin 0 holds the largest logits
  // weights vanish beyond (max - l)/T > 27.73, so the bins cover 28 T logit units
  const float scale_a = (float)SMP_BINS / (28.f * temperature);
  for (int i = tid; i < SMP_BINS; i += SMP_THREADS) { sh.hist[i] = 0ull; sh.cnt[i] = 0u; }
  if (tid == 0) { sh.carried = 0ull; sh.kmin = 0xffffffffu; sh.kmax = 0u; sh.n_cand = 0u; sh.tie_max_id = 0x7fffffff; }
  __syncthreads();
  unsigned long long mysum = 0ull;
  SMP_FOREACH({
    (void)i;
    const unsigned long long w = smp_weight(x, mx, inv_t_log2e);
    if (w) {
      smp_hist_add(&sh.hist[min(SMP_BINS - 1, (int)((mx - x) * scale_a))], w);
      mysum += w;
    }
  })
  block_excl_scan_u64(mysum, sh.wtot, &sh.loc_total);
  cluster.sync();                                  // every slice's histogram and total are complete
  unsigned long long cut = 0ull;
  if (rank == 0) {
    unsigned long long total = 0ull;
#pragma unroll
    for (int k = 0; k < SMP_MAX_CLUSTER; ++k)
      if (k < SMP_CLUSTER) total += peer[k]->loc_total;
    for (int i = tid; i < SMP_BINS; i += SMP_THREADS) {
      unsigned long long h = sh.hist[i];
#pragma unroll
      for (int k = 1; k < SMP_MAX_CLUSTER; ++k)
        if (k < SMP_CLUSTER) h += peer[k]->hist[i];
      sh.hist[i] = h;
    }
    __syncthreads();
    cut = __double2ull_rd((double)a.top_p[r] * (double)total);
    if (cut > total) cut = total;
    smp_select_bin(sh, cut, false);
    if (tid == 0) sh.bc_bin = sh.sel_bin;
  }
  cluster.sync();
  const int bin_a = peer[0]->bc_bin;

  // ---- the tokens of the selected bin in this slice, with their key range
  SMP_FOREACH({
    if (min(SMP_BINS - 1, (int)((mx - x) * scale_a)) == bin_a) {
      const unsigned int c = atomicAdd(&sh.n_cand, 1u);
      if (c < (unsigned)SMP_CAND) { sh.cand_x[c] = x; sh.cand_id[c] = i; }
      const uint32_t k = ordered_key(x);
      atomicMin(&sh.kmin, k);
      atomicMax(&sh.kmax, k);
    }
  })
  cluster.sync();                                  // every slice's candidates are listed
  if (rank == 0) {
    // gather the other slices' candidates behind this slice's
    unsigned int n_all = sh.n_cand, kmin = sh.kmin, kmax = sh.kmax;
    unsigned int off[SMP_MAX_CLUSTER];
    off[0] = 0u;
#pragma unroll
    for (int k = 1; k < SMP_MAX_CLUSTER; ++k) {
      if (k >= SMP_CLUSTER) break;
      off[k] = n_all;
      n_all += peer[k]->n_cand;
      kmin = min(kmin, peer[k]->kmin);
      kmax = max(kmax, peer[k]->kmax);
    }
    __syncthreads();                               // everyone has read n_cand / kmin / kmax of this CTA
    const int n_cand = (int)n_all;
    if (tid == 0) { sh.sel_cnt = n_all; sh.bc_overflow = n_cand > SMP_CAND ? 1 : 0; }   // sel_cnt stands if no refinement is needed
    if (n_cand <= SMP_CAND) {
#pragma unroll
      for (int k = 1; k < SMP_MAX_CLUSTER; ++k) {
        if (k >= SMP_CLUSTER) break;
        const int nk = (int)(k + 1 < SMP_CLUSTER ? off[k + 1] : n_all) - (int)off[k];
        for (int c = tid; c < nk; c += SMP_THREADS) {
          sh.cand_x[off[k] + c] = peer[k]->cand_x[c];
          sh.cand_id[off[k] + c] = peer[k]->cand_id[c];
        }
      }
    }
    __syncthreads();
    if (n_cand > SMP_CAND) {
      // rare: this CTA finishes the row alone, reading all of it
      smp_tail_full_row(sh, a, r, lg, mx, inv_t_log2e, scale_a, bin_a, cut, u24);
    } else {
      // ---- exact refinement in key space, over the candidates only, until one key remains
      for (int pass = 0; pass < 4 && kmax > kmin; ++pass) {
        const unsigned long long width = (unsigned long long)(kmax - kmin) + 1ull;
        __syncthreads();
        for (int i = tid; i < SMP_BINS; i += SMP_THREADS) { sh.hist[i] = 0ull; sh.cnt[i] = 0u; }
        __syncthreads();
        for (int c = tid; c < n_cand; c += SMP_THREADS) {
          const float x = sh.cand_x[c];
          const uint32_t k = ordered_key(x);
          if (k >= kmin && k <= kmax) {
            const int bin = smp_key_bin(k, kmin, width);
            atomicAdd(&sh.hist[bin], smp_weight(x, mx, inv_t_log2e));
            atomicAdd(&sh.cnt[bin], 1u);
          }
        }
        __syncthreads();
        smp_select_bin(sh, cut, true);
        const KeyRange kr = smp_narrow(sh, kmin, width);
        kmin = kr.kmin; kmax = kr.kmax;
      }
      __syncthreads();
      // Now every token with key == kmin (== kmax) is tied at the nucleus edge.
      const uint32_t kstar = kmin;
      const unsigned long long carried = sh.carried;     // weight of tokens with key > kstar
      const unsigned int n_tied = sh.sel_cnt;
      const unsigned long long wstar = n_tied ? sh.sel_sum / n_tied : 0ull;
      unsigned long long m_ties = 1ull;
      if (wstar > 0ull && cut > carried) m_ties = (cut - carried + wstar - 1ull) / wstar;
      if (m_ties < 1ull) m_ties = 1ull;
      if (m_ties > n_tied) m_ties = n_tied;
      const unsigned long long Z = carried + m_ties * wstar;
      // the tied tokens that belong to the nucleus are the m_ties lowest ids: find the largest of them
      if (m_ties < n_tied) {
        for (int c = tid; c < n_cand; c += SMP_THREADS) {
          if (ordered_key(sh.cand_x[c]) != kstar) continue;
          const int id = sh.cand_id[c];
          unsigned long long rank_ = 0ull;
          for (int j = 0; j < n_cand; ++j)
            rank_ += (ordered_key(sh.cand_x[j]) == kstar && sh.cand_id[j] < id) ? 1ull : 0ull;
          if (rank_ == m_ties - 1ull) sh.tie_max_id = id;
        }
      }
      __syncthreads();
      if (tid == 0) {
        sh.bc_kstar = kstar;
        sh.bc_wstar = wstar;
        sh.bc_tie_max_id = sh.tie_max_id;
        sh.bc_rdraw = __umul64hi(Z, (unsigned long long)u24 << 40);   // floor(u24 * Z / 2^24)
      }
    }
  }
  cluster.sync();
  if (peer[0]->bc_overflow) {
    cluster.sync();
    return;
  }
  const uint32_t kstar = peer[0]->bc_kstar;
  const unsigned long long wstar = peer[0]->bc_wstar, rdraw = peer[0]->bc_rdraw;
  const int tie_max_id = peer[0]->bc_tie_max_id;

  // ---- inverse CDF over the nucleus in ascending id order.  Inside the slice warp w owns a contiguous
  // range of units and its lanes take consecutive units, so ids ascend with the lane in every step.
  const int per_warp = (u_hi - u_lo + 31) / 32;
  const int w_begin = min(u_hi, u_lo + warp * per_warp), w_end = min(u_hi, w_begin + per_warp);
  const int n_it = (per_warp + 31) / 32;                // the same for every warp
  auto unit_weights = [&](int u, unsigned long long (&w)[4]) {
    float xs[4];
    int cntu = 1;
    if (vec) {
      const float4 q = reinterpret_cast<const float4 *>(lg)[u];
      xs[0] = q.x; xs[1] = q.y; xs[2] = q.z; xs[3] = q.w;
      cntu = 4;
    } else {
      xs[0] = lg[u];
    }
    const int id0 = vec ? 4 * u : u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      w[j] = 0ull;
      if (j < cntu) {
        const uint32_t k = ordered_key(xs[j]);
        if (k > kstar) w[j] = smp_weight(xs[j], mx, inv_t_log2e);
        else if (k == kstar && id0 + j <= tie_max_id) w[j] = wstar;
      }
    }
  };
  unsigned long long ws = 0ull;
  for (int it = 0; it < n_it; ++it) {
    const int u = w_begin + it * 32 + lane;
    if (u < w_end) {
      unsigned long long w[4];
      unit_weights(u, w);
      ws += w[0] + w[1] + w[2] + w[3];
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
  if (lane == 0) sh.loc_wtot[warp] = ws;
  cluster.sync();                                  // every slice's warp totals are in place
  if (rank == 0 && warp < SMP_CLUSTER) {
    // warp k scans the 32 warp totals of slice k; lane 0 of warp 0 then walks the four slice totals
    const unsigned long long w = peer[warp]->loc_wtot[lane];
    unsigned long long inc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    sh.hist[warp * 32 + lane] = inc - w;           // weight before the warp inside its slice (hist is free by now)
    if (lane == 31) sh.wtot[warp] = inc;           // slice total
  }
  __syncthreads();
  if (rank == 0 && tid == 0) {
    unsigned long long before = 0ull;
    int sr = SMP_CLUSTER - 1, sw = 31;
    bool found = false;
    for (int k = 0; k < SMP_CLUSTER && !found; ++k) {
      if (rdraw < before + sh.wtot[k]) {
        const unsigned long long inside = rdraw - before;
        sr = k;
        sw = 31;
        for (int w = 0; w < 32; ++w) {
          const unsigned long long b0 = sh.hist[k * 32 + w];
          const unsigned long long b1 = w < 31 ? sh.hist[k * 32 + w + 1] : sh.wtot[k];
          if (inside >= b0 && inside < b1) { sw = w; break; }
        }
        before += sh.hist[k * 32 + sw];
        found = true;
      } else {
        before += sh.wtot[k];
      }
    }
    sh.bc_sel_rank = sr; sh.bc_sel_warp = sw; sh.bc_before = before;
  }
  cluster.sync();
  const int sel_rank = peer[0]->bc_sel_rank, sel_warp = peer[0]->bc_sel_warp;
  unsigned long long run = peer[0]->bc_before;
  if (rank == sel_rank && warp == sel_warp) {
    int tok = (vec ? 4 * w_end : w_end) - 1;
    for (int it = 0; it < n_it; ++it) {
      const int u = w_begin + it * 32 + lane;
      unsigned long long w[4] = {0ull, 0ull, 0ull, 0ull};
      if (u < w_end) unit_weights(u, w);
      const unsigned long long s_ = w[0] + w[1] + w[2] + w[3];
      unsigned long long inc = s_;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, run + inc > rdraw);
      if (hit) {
        const int Lh = __ffs(hit) - 1;
        if (lane == Lh) {
          unsigned long long c = run + inc - s_;
          const int id0 = vec ? 4 * u : u;
          int t = id0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            c += w[j];
            if (c > rdraw) { t = id0 + j; break; }
          }
          tok = t;
        }
        tok = __shfl_sync(0xffffffffu, tok, Lh);
        break;
      }
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) a.out_token[r] = tok;
  }
  cluster.sync();                                  // nobody leaves while its shared memory may still be read
}
#undef SMP_FOREACH

// ---------------------------------------------------------------- decode bookkeeping
// active_mask / seeds_in are the step's inputs in PINNED HOST memory, read here through their device mapping:
// 9 bytes per slot cross the bus inside this kernel instead of in two copy nodes in front of it.
// The rows of the step are the slots in a new order: the slots with a request this step first (ascending slot), the
// others behind them.  Which row a request lands in depends on its co-tenants; no value of the step depends on the
// row (that is the invariance the whole path is built for), and with the requests in the first rows the GEMMs can
// leave out whole blocks of rows that hold none (row_blocks: bit b = block b holds a request; blocks of 64 rows up
// to 128 padded rows, of 128 rows above).  Per-slot sampling state is copied to the row's place.  One CTA.
__global__ void __launch_bounds__(256) prepare_rows_kernel(const uint8_t *active_mask, const uint64_t *seeds_in, uint64_t *seeds_out,
                                                           const int *in_use, const int *ctx_len, const int *pending,
                                                           const float *temp, const float *top_p, const int *step, int B,
                                                           int *row_token, int *row_pos, int *row_active, int *row_slot,
                                                           int *do_sample, float *row_temp, float *row_top_p, int *row_step,
                                                           int *slot_row, int *row_blocks) {
  griddep_launch_dependents();
  griddep_wait();
  __shared__ int warp_cnt[8];
  const int s = threadIdx.x, lane = s & 31, warp = s >> 5;
  const int act = (s < B && active_mask[s] != 0 && in_use[s] != 0) ? 1 : 0;
  const unsigned m = __ballot_sync(0xffffffffu, act != 0);
  if (lane == 0) warp_cnt[warp] = __popc(m);
  __syncthreads();
  int before = __popc(m & ((1u << lane) - 1u)), n_act = 0;
  for (int w = 0; w < 8; ++w) {
    if (w < warp) before += warp_cnt[w];
    n_act += warp_cnt[w];
  }
  if (s == 0 && row_blocks) {
    const int blk = B <= 128 ? 64 : 128;
    *row_blocks = (n_act > 0 ? 1 : 0) | (n_act > blk ? 2 : 0);
  }
  if (s >= B) return;
  const int r = act ? before : n_act + (s - before);   // requests first, in slot order; then the other slots
  slot_row[s] = r;
  row_slot[r] = s;
  row_active[r] = act;
  row_pos[r] = act ? ctx_len[s] : 0;
  row_token[r] = act ? pending[s] : 0;
  do_sample[r] = act;
  seeds_out[r] = seeds_in[s];
  row_temp[r] = temp[s];
  row_top_p[r] = top_p[s];
  row_step[r] = step[s];
}

// out_tokens / status_out are PINNED HOST memory written through their device mapping (the step's results: 4
// bytes per slot and the status word), fenced system-wide; the host reads them after synchronising the stream.
__global__ void advance_kernel(const int *slot_row, const int *row_active, const int *sampled, int B, int *ctx_len, int *step,
                               int *pending, int *out_tokens, const int *status_in, int *status_out) {
  griddep_launch_dependents();
  griddep_wait();
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s == 0) *status_out = *status_in;
  if (s >= B) { __threadfence_system(); return; }
  const int r = slot_row[s];
  if (row_active[r]) {
    const int tok = sampled[r];
    pending[s] = tok;
    ctx_len[s] += 1;
    step[s] += 1;
    out_tokens[s] = tok;
  } else {
    out_tokens[s] = -1;
  }
  __threadfence_system();
}

__global__ void kv_copy_kernel(KvLayout kv, int layer, int slot, int pos0, int n, float *k, float *v, int write) {
  const int KD = kv.n_kv * kv.hd;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)n * KD) return;
  const int t = (int)(idx / KD), e = (int)(idx - (size_t)t * KD);
  const int g = e / kv.hd, i = e - g * kv.hd;
  const int pos = pos0 + t;
  const int blk = kv.block_table[(size_t)slot * kv.max_blocks + pos / KV_BLOCK];
  __half *base = kv.pool + (size_t)layer * kv.layer_stride + (size_t)blk * 2 * kv.n_kv * KV_BLOCK * kv.hd;
  __half *kp = base + kv_k_off(kv.hd, g, pos % KV_BLOCK, i);
  __half *vp = base + kv_v_off(kv.n_kv, kv.hd, g, pos % KV_BLOCK, i);
  if (write) {
    *kp = __float2half_rn(k[idx]);
    *vp = __float2half_rn(v[idx]);
  } else {
    k[idx] = __half2float(*kp);
    v[idx] = __half2float(*vp);
  }
}

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Synthetic cache contents for timing runs: position-hashed normals, one thread per (layer, token, pair).
__global__ void kv_fill_kernel(KvLayout kv, int n_layers, int slot, int n, float std, uint64_t seed) {
  const int KD = kv.n_kv * kv.hd;
  const size_t per_layer = (size_t)n * KD;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= per_layer * n_layers) return;
  const int layer = (int)(idx / per_layer);
  const size_t rem = idx - (size_t)layer * per_layer;
  const int t = (int)(rem / KD), e = (int)(rem - (size_t)t * KD);
  const int g = e / kv.hd, i = e - g * kv.hd;
  const uint64_t h = mix64(seed ^ mix64(((uint64_t)slot << 48) ^ ((uint64_t)layer << 40) ^ ((uint64_t)t << 16) ^ (uint64_t)e));
  const float u1 = ((float)(uint32_t)(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
  const float u2 = (float)(uint32_t)((h >> 8) & 0xFFFFFFu) * (1.0f / 16777216.0f);
  const float rad = sqrtf(-2.0f * logf(u1)) * std;
  const int blk = kv.block_table[(size_t)slot * kv.max_blocks + t / KV_BLOCK];
  __half *base = kv.pool + (size_t)layer * kv.layer_stride + (size_t)blk * 2 * kv.n_kv * KV_BLOCK * kv.hd;
  base[kv_k_off(kv.hd, g, t % KV_BLOCK, i)] = __float2half_rn(rad * cospif(2.0f * u2));
  base[kv_v_off(kv.n_kv, kv.hd, g, t % KV_BLOCK, i)] = __float2half_rn(rad * sinpif(2.0f * u2));
}

}  // namespace

cudaError_t launch_resid_norm(float *h, int H, const __nv_bfloat16 *embed, const Rows &rows, const GemmOut *prev,
                              const __nv_bfloat16 *gains, float eps, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                              cudaStream_t st) {
  GemmOut g{};
  if (prev) g = *prev;
  int threads = H / 4;
  if (threads > NORM_MAX_THREADS) threads = NORM_MAX_THREADS;
  threads = (threads + 31) / 32 * 32;
  return launch_k(resid_norm_kernel, dim3(rows.R), dim3(threads), 0, st, true, h, H, embed, rows, g, prev ? 0 : 1, gains,
                  eps, out_hi, out_lo);
}

cudaError_t launch_qkv_post(const GemmOut &qkv, const Rows &rows, const float2 *rope_tab, int nq, const KvLayout &kv,
                            int layer, float *q_out, int *d_status, cudaStream_t st) {
  return launch_k(qkv_post_kernel, dim3(nq + 2 * kv.n_kv, rows.R), dim3(kv.hd / 2), 0, st, true, qkv, rows, rope_tab, nq,
                  kv, layer, q_out, d_status);
}

cudaError_t launch_swiglu(const GemmOut &gu, int R, int F, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, cudaStream_t st) {
  return launch_k(swiglu_kernel, dim3((F / 4 + 255) / 256, R), dim3(256), 0, st, true, gu, F, out_hi, out_lo);
}

cudaError_t launch_split(const float *x, int R, int K, __nv_bfloat16 *hi, __nv_bfloat16 *lo, cudaStream_t st) {
  const size_t n = (size_t)R * K;
  split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(x, n, hi, lo);
  return cudaGetLastError();
}

cudaError_t launch_sampler(const SampleArgs &a, int R, cudaStream_t st, bool pdl) {
  // CTAs per row: more CTAs shorten a row's passes, fewer keep all rows' clusters resident at once (two CTAs per SM:
  // 296 in all).  Measured (vocabulary 151 936; 2 / 3 / 4 / 5 / 6 / 7 CTAs per row): 40 sampled rows 90.8 / 70.2 / 85.6 /
  // 73.1 / 72.1 / 98.1 us, 64 rows 90.5 / 101.2 / 89.0 / 111.8 / 111.6 / 124.3 us, 128 rows 141.0 / 153.9 / 165.2 / 175.5 /
  // 193.2 / 226.5 us.  The launch shape is fixed in the step's graph, so it follows the padded row count.
  int nc = R <= 16 ? 6 : R <= 64 ? 3 : 2;
  if (const char *c = getenv("CORUN_SAMPLER_CLUSTER")) {   // (timing experiments)
    const int v = atoi(c);
    if (v >= 1 && v <= SMP_MAX_CLUSTER) nc = v;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(R * nc);
  cfg.blockDim = dim3(SMP_THREADS);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = nc;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pdl && g_use_pdl) ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, sampler_kernel, a);
}

cudaError_t launch_prepare_rows(const uint8_t *active_mask, const uint64_t *seeds_in, uint64_t *seeds_out, const int *in_use,
                                const int *ctx_len, const int *pending, const float *temp, const float *top_p, const int *step,
                                int B, int *row_token, int *row_pos, int *row_active, int *row_slot, int *do_sample,
                                float *row_temp, float *row_top_p, int *row_step, int *slot_row, int *row_blocks,
                                cudaStream_t st) {
  if (B > 256) return cudaErrorInvalidValue;
  prepare_rows_kernel<<<1, 256, 0, st>>>(active_mask, seeds_in, seeds_out, in_use, ctx_len, pending, temp, top_p, step, B,
                                         row_token, row_pos, row_active, row_slot, do_sample, row_temp, row_top_p, row_step,
                                         slot_row, row_blocks);
  return cudaGetLastError();
}

cudaError_t launch_advance(const int *slot_row, const int *row_active, const int *sampled, int B, int *ctx_len, int *step,
                           int *pending, int *out_tokens, const int *status_in, int *status_out, cudaStream_t st) {
  return launch_k(advance_kernel, dim3((B + 127) / 128), dim3(128), 0, st, true, slot_row, row_active, sampled, B, ctx_len,
                  step, pending, out_tokens, status_in, status_out);
}

cudaError_t launch_kv_copy(const KvLayout &kv, int layer, int slot, int pos0, int n, float *k, float *v, int write,
                           cudaStream_t st) {
  const size_t tot = (size_t)n * kv.n_kv * kv.hd;
  if (tot == 0) return cudaSuccess;
  kv_copy_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(kv, layer, slot, pos0, n, k, v, write);
  return cudaGetLastError();
}

cudaError_t launch_kv_fill(const KvLayout &kv, int n_layers, int slot, int n, float std, uint64_t seed, cudaStream_t st) {
  const size_t tot = (size_t)n * kv.n_kv * kv.hd * n_layers;
  if (tot == 0) return cudaSuccess;
  kv_fill_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(kv, n_layers, slot, n, std, seed);
  return cudaGetLastError();
}

cudaError_t launch_variate(uint64_t seed, uint64_t t, uint32_t *out, cudaStream_t st) {
  variate_kernel<<<1, 1, 0, st>>>(seed, t, out);
  return cudaGetLastError();
}

}  // namespace corun
