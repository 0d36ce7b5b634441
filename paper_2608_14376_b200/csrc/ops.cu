// Non-GEMM kernels of the row program: residual + RMSNorm, RoPE + KV append,
// request-local split-KV paged attention with a fixed-order combine, SwiGLU,
// seeded sampling, decode bookkeeping.  Every reduction has one fixed order
// that depends on the row's own data and the model shape only; no float atomics.
#include "ops.cuh"

#include <math_constants.h>

namespace corun {

namespace {

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// Sum over the block in a fixed order: xor-butterfly inside each warp, then
// the warp totals added in ascending warp order by every thread.
template <int NWARPS>
__device__ __forceinline__ float block_sum_fixed(float v, float *scratch /*[NWARPS]*/) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < NWARPS; ++w) t += scratch[w];
  return t;
}

// ---------------------------------------------------------------- residual + RMSNorm
constexpr int NORM_THREADS = 256;

__global__ void __launch_bounds__(NORM_THREADS)
resid_norm_kernel(float *__restrict__ h, int H, const __nv_bfloat16 *__restrict__ embed, Rows rows, GemmOut prev,
                  int first, const __nv_bfloat16 *__restrict__ gains, float eps, __nv_bfloat16 *__restrict__ out_hi,
                  __nv_bfloat16 *__restrict__ out_lo) {
  __shared__ float scratch[NORM_THREADS / 32];
  const int r = blockIdx.x;
  float *hr = h + (size_t)r * H;
  float ss = 0.f;
  if (first) {
    const __nv_bfloat16 *e = embed + (size_t)rows.token[r] * H;
    for (int i = threadIdx.x; i < H; i += NORM_THREADS) {
      const float x = __bfloat162float(e[i]);
      hr[i] = x;
      ss = fmaf(x, x, ss);
    }
  } else {
    for (int i = threadIdx.x; i < H; i += NORM_THREADS) {
      const float x = hr[i] + gemm_load(prev, r, i);
      hr[i] = x;
      ss = fmaf(x, x, ss);
    }
  }
  const float tot = block_sum_fixed<NORM_THREADS / 32>(ss, scratch);
  const float inv = rsqrtf(tot / (float)H + eps);
  for (int i = threadIdx.x; i < H; i += NORM_THREADS) {
    const float y = hr[i] * inv * __bfloat162float(gains[i]);
    __nv_bfloat16 a, b;
    split_bf16(y, a, b);
    out_hi[(size_t)r * H + i] = a;
    out_lo[(size_t)r * H + i] = b;
  }
}

// ---------------------------------------------------------------- RoPE + KV append
__global__ void __launch_bounds__(256)
qkv_post_kernel(GemmOut qkv, Rows rows, const float2 *__restrict__ rope_tab, int nq, KvLayout kv, int layer,
                float *__restrict__ q_out) {
  const int r = blockIdx.x;
  const int hd = kv.hd, half = hd >> 1, nkv = kv.n_kv;
  const int pos = rows.pos[r];
  const int active = rows.active[r];
  const float2 *cs = rope_tab + (size_t)pos * half;
  const int QD = nq * hd, KD = nkv * hd;
  __half *kdst = nullptr, *vdst = nullptr;
  if (active) {
    const int blk = kv.block_table[(size_t)rows.slot[r] * kv.max_blocks + pos / KV_BLOCK];
    __half *base = kv.pool + (size_t)layer * kv.layer_stride + (size_t)blk * 2 * nkv * KV_BLOCK * hd;
    kdst = base + (size_t)(pos % KV_BLOCK) * hd;                       // + g * 16 * hd per head
    vdst = base + (size_t)nkv * KV_BLOCK * hd + (size_t)(pos % KV_BLOCK) * hd;
  }
  // rotated pairs of q and k
  const int n_pairs = (nq + nkv) * half;
  for (int idx = threadIdx.x; idx < n_pairs; idx += blockDim.x) {
    const int head = idx / half, i = idx - head * half;
    const int col = head * hd + i;                 // q heads then k heads are contiguous in the GEMM output
    const float a = gemm_load(qkv, r, col), b = gemm_load(qkv, r, col + half);
    const float2 t = cs[i];                        // (cos, sin)
    const float ra = a * t.x - b * t.y, rb = a * t.y + b * t.x;
    if (head < nq) {
      q_out[(size_t)r * QD + col] = ra;
      q_out[(size_t)r * QD + col + half] = rb;
    } else if (active) {
      const int g = head - nq;
      kdst[(size_t)g * KV_BLOCK * hd + i] = __float2half_rn(ra);
      kdst[(size_t)g * KV_BLOCK * hd + i + half] = __float2half_rn(rb);
    }
  }
  if (active) {
    for (int idx = threadIdx.x; idx < KD; idx += blockDim.x) {
      const int g = idx / hd, i = idx - g * hd;
      vdst[(size_t)g * KV_BLOCK * hd + i] = __float2half_rn(gemm_load(qkv, r, QD + KD + idx));
    }
  }
}

// ---------------------------------------------------------------- split-KV paged attention
constexpr int ATT_THREADS = 128;

template <int HD, int GROUP>
__global__ void __launch_bounds__(ATT_THREADS)
attn_split_kernel(const float *__restrict__ q, Rows rows, int nq, KvLayout kv, int layer, int max_splits,
                  float *__restrict__ part_acc, float *__restrict__ part_ml) {
  constexpr int CH = HD / 8;                 // 16-byte chunks per cached row
  constexpr int NTG = ATT_THREADS / CH;      // token groups in the value pass
  const int split = blockIdx.x, g = blockIdx.y, r = blockIdx.z;
  if (!rows.active[r]) return;
  const int ctx = rows.pos[r] + 1;           // the new token attends to itself too
  const int t0 = split * ATT_SPLIT;
  if (t0 >= ctx) return;
  const int ntok = min(ATT_SPLIT, ctx - t0);

  __shared__ __align__(16) float q_s[GROUP][HD];
  __shared__ __align__(16) float p_s[ATT_SPLIT * GROUP];
  __shared__ __align__(16) float red_s[NTG][GROUP][HD];
  __shared__ float wred_s[ATT_THREADS / 32][GROUP];
  __shared__ int blk_s[ATT_SPLIT / KV_BLOCK];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nkv = kv.n_kv;
  const __half *pool = kv.pool + (size_t)layer * kv.layer_stride;
  const size_t blk_halfs = (size_t)2 * nkv * KV_BLOCK * HD;
  // 1/sqrt(hd) * log2(e): scores live in the base-2 domain
  const float qscale = (HD == 128 ? 0.08838834764831845f : 0.125f) * 1.4426950408889634f;
  for (int i = tid; i < GROUP * HD; i += ATT_THREADS)
    q_s[i / HD][i % HD] = q[(size_t)r * nq * HD + (size_t)(g * GROUP) * HD + i] * qscale;
  if (tid < ATT_SPLIT / KV_BLOCK) {
    const int b = t0 / KV_BLOCK + tid;
    blk_s[tid] = (b * KV_BLOCK < ctx) ? kv.block_table[(size_t)rows.slot[r] * kv.max_blocks + b] : 0;
  }
  __syncthreads();

  // ---- scores: one thread per cached token, dot product in ascending dim order
  float lmax[GROUP];
#pragma unroll
  for (int h = 0; h < GROUP; ++h) lmax[h] = -CUDART_INF_F;
#pragma unroll
  for (int rep = 0; rep < ATT_SPLIT / ATT_THREADS; ++rep) {
    const int tt = tid + rep * ATT_THREADS;
    float s[GROUP];
#pragma unroll
    for (int h = 0; h < GROUP; ++h) s[h] = 0.f;
    if (tt < ntok) {
      const uint4 *kp = reinterpret_cast<const uint4 *>(pool + (size_t)blk_s[tt / KV_BLOCK] * blk_halfs +
                                                        (size_t)g * KV_BLOCK * HD + (size_t)(tt % KV_BLOCK) * HD);
#pragma unroll 4
      for (int c = 0; c < CH; ++c) {
        const uint4 kk = __ldg(kp + c);
        const __half2 *k2 = reinterpret_cast<const __half2 *>(&kk);
        float kf[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __half22float2(k2[j]);
          kf[2 * j] = f.x;
          kf[2 * j + 1] = f.y;
        }
#pragma unroll
        for (int h = 0; h < GROUP; ++h) {
          const float4 qa = *reinterpret_cast<const float4 *>(&q_s[h][c * 8]);
          const float4 qb = *reinterpret_cast<const float4 *>(&q_s[h][c * 8 + 4]);
          float a = s[h];
          a = fmaf(qa.x, kf[0], a); a = fmaf(qa.y, kf[1], a); a = fmaf(qa.z, kf[2], a); a = fmaf(qa.w, kf[3], a);
          a = fmaf(qb.x, kf[4], a); a = fmaf(qb.y, kf[5], a); a = fmaf(qb.z, kf[6], a); a = fmaf(qb.w, kf[7], a);
          s[h] = a;
        }
      }
#pragma unroll
      for (int h = 0; h < GROUP; ++h) lmax[h] = fmaxf(lmax[h], s[h]);
    } else {
#pragma unroll
      for (int h = 0; h < GROUP; ++h) s[h] = -CUDART_INF_F;
    }
#pragma unroll
    for (int h = 0; h < GROUP; ++h) p_s[tt * GROUP + h] = s[h];
  }
  // ---- split maximum (exact, order-free)
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    float v = lmax[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (lane == 0) wred_s[warp][h] = v;
  }
  __syncthreads();
  float m[GROUP], lsum[GROUP];
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    float v = wred_s[0][h];
#pragma unroll
    for (int w = 1; w < ATT_THREADS / 32; ++w) v = fmaxf(v, wred_s[w][h]);
    m[h] = v;
    lsum[h] = 0.f;
  }
  __syncthreads();
  // ---- probabilities and their sum (fixed tree)
#pragma unroll
  for (int rep = 0; rep < ATT_SPLIT / ATT_THREADS; ++rep) {
    const int tt = tid + rep * ATT_THREADS;
#pragma unroll
    for (int h = 0; h < GROUP; ++h) {
      const float p = exp2f(p_s[tt * GROUP + h] - m[h]);   // -inf -> 0 for the tail
      p_s[tt * GROUP + h] = p;
      lsum[h] += p;
    }
  }
#pragma unroll
  for (int h = 0; h < GROUP; ++h) {
    float v = lsum[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) wred_s[warp][h] = v;
  }
  __syncthreads();
  if (tid < GROUP) {
    float v = 0.f;
    for (int w = 0; w < ATT_THREADS / 32; ++w) v += wred_s[w][tid];
    float *ml = part_ml + (((size_t)r * nq + g * GROUP + tid) * max_splits + split) * 2;
    ml[0] = m[tid];
    ml[1] = v;
  }
  // ---- weighted values: thread = (8-dim chunk, token group), tokens ascending inside a group
  const int dc = tid % CH, tg = tid / CH;
  float acc[GROUP][8];
#pragma unroll
  for (int h = 0; h < GROUP; ++h)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[h][j] = 0.f;
  for (int tt = tg; tt < ntok; tt += NTG) {
    const uint4 *vp = reinterpret_cast<const uint4 *>(pool + (size_t)blk_s[tt / KV_BLOCK] * blk_halfs +
                                                      (size_t)(nkv + g) * KV_BLOCK * HD + (size_t)(tt % KV_BLOCK) * HD);
    const uint4 vv = __ldg(vp + dc);
    const __half2 *v2 = reinterpret_cast<const __half2 *>(&vv);
    float vf[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(v2[j]);
      vf[2 * j] = f.x;
      vf[2 * j + 1] = f.y;
    }
#pragma unroll
    for (int h = 0; h < GROUP; ++h) {
      const float p = p_s[tt * GROUP + h];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[h][j] = fmaf(p, vf[j], acc[h][j]);
    }
  }
#pragma unroll
  for (int h = 0; h < GROUP; ++h)
#pragma unroll
    for (int j = 0; j < 8; ++j) red_s[tg][h][dc * 8 + j] = acc[h][j];
  __syncthreads();
  for (int idx = tid; idx < GROUP * HD; idx += ATT_THREADS) {
    const int h = idx / HD, d = idx - h * HD;
    float o = 0.f;
#pragma unroll
    for (int t = 0; t < NTG; ++t) o += red_s[t][h][d];
    part_acc[(((size_t)r * nq + g * GROUP + h) * max_splits + split) * HD + d] = o;
  }
}

// Combines the splits of each (row, head) in ascending split order.
__global__ void __launch_bounds__(256)
attn_combine_kernel(Rows rows, int nq, int hd, int max_splits, const float *__restrict__ part_acc,
                    const float *__restrict__ part_ml, __nv_bfloat16 *__restrict__ out_hi,
                    __nv_bfloat16 *__restrict__ out_lo) {
  const int r = blockIdx.x;
  const int QD = nq * hd;
  const bool active = rows.active[r] != 0;
  const int nsplit = active ? (rows.pos[r] + 1 + ATT_SPLIT - 1) / ATT_SPLIT : 0;
  for (int idx = threadIdx.x; idx < QD; idx += blockDim.x) {
    float o = 0.f;
    if (active) {
      const int j = idx / hd, d = idx - j * hd;
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
    __nv_bfloat16 a, b;
    split_bf16(o, a, b);
    out_hi[(size_t)r * QD + idx] = a;
    out_lo[(size_t)r * QD + idx] = b;
  }
}

// ---------------------------------------------------------------- SwiGLU
__global__ void __launch_bounds__(256)
swiglu_kernel(GemmOut gu, int F, __nv_bfloat16 *__restrict__ out_hi, __nv_bfloat16 *__restrict__ out_lo) {
  const int r = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= F) return;
  const float g = gemm_load(gu, r, i), u = gemm_load(gu, r, F + i);
  const float y = g / (1.f + expf(-g)) * u;
  __nv_bfloat16 a, b;
  split_bf16(y, a, b);
  out_hi[(size_t)r * F + i] = a;
  out_lo[(size_t)r * F + i] = b;
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

struct SmpShared {
  unsigned long long hist[SMP_BINS];
  unsigned int cnt[SMP_BINS];
  unsigned long long wtot[32];
  unsigned long long total, carried, sel_sum;
  float red_val[32];
  int red_idx[32];
  unsigned int kmin, kmax, sel_cnt;
  int sel_bin, winner;
};

// Integer weight of a token: floor(2^40 * exp2(x)), x = fl32(fl32(l - max) * inv_t_log2e).
// exp2 is spelled out so that the integer is the same on every IEEE-754 machine:
// x = n + f with n = rint(x); degree-7 Taylor polynomial of 2^f (ln(2)^k / k! in fp32),
// Horner form, separately rounded multiplies and adds; exact scaling by 2^(n+40).
__device__ __forceinline__ unsigned long long smp_weight(float l, float mx, float inv_t_log2e) {
  const float x = __fmul_rn(__fsub_rn(l, mx), inv_t_log2e);
  if (!(x > -64.0f)) return 0ull;
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

// After a histogram pass: finds the first bin (ascending index = descending
// logit) that is non-empty and whose running weight reaches the cut; adds the
// weight of the bins before it to `carried`.
__device__ void smp_select_bin(SmpShared &sh, unsigned long long cut) {
  const int tid = threadIdx.x;
  const unsigned long long a = sh.hist[2 * tid], b = sh.hist[2 * tid + 1];
  unsigned long long tot;
  const unsigned long long before = block_excl_scan_u64(a + b, sh.wtot, &tot);
  if (tid == 0) sh.sel_bin = SMP_BINS;
  __syncthreads();
  const unsigned long long base = sh.carried + before;
  if (sh.cnt[2 * tid] && base + a >= cut) atomicMin(&sh.sel_bin, 2 * tid);
  else if (sh.cnt[2 * tid + 1] && base + a + b >= cut) atomicMin(&sh.sel_bin, 2 * tid + 1);
  __syncthreads();
  const int sel = sh.sel_bin;   // < SMP_BINS: total weight always reaches the cut
  if (sel < SMP_BINS && (sel >> 1) == tid) {
    sh.carried = base + ((sel & 1) ? a : 0ull);
    sh.sel_sum = (sel & 1) ? b : a;
    sh.sel_cnt = sh.cnt[sel];
  }
  __syncthreads();
}

__global__ void __launch_bounds__(SMP_THREADS) sampler_kernel(SampleArgs a) {
  const int r = blockIdx.x;
  if (!a.do_sample[r]) return;
  __shared__ SmpShared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = a.V;
  const float *lg = a.logits + (size_t)r * V;

  // ---- argmax, lowest id on ties
  float bv = -CUDART_INF_F;
  int bi = 0x7fffffff;
  for (int i = tid; i < V; i += SMP_THREADS) {
    const float x = lg[i];
    if (x > bv || (x == bv && i < bi)) { bv = x; bi = i; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if (lane == 0) { sh.red_val[warp] = bv; sh.red_idx[warp] = bi; }
  __syncthreads();
  bv = sh.red_val[0]; bi = sh.red_idx[0];
  for (int w = 1; w < SMP_THREADS / 32; ++w) {
    const float ov = sh.red_val[w];
    const int oi = sh.red_idx[w];
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  const float temperature = a.temperature[r];
  if (!(temperature > 0.f)) {
    if (tid == 0) a.out_token[r] = bi;
    return;
  }
  const float mx = bv;
  const float inv_t_log2e = __fdiv_rn(0x1.715476p+0f, temperature);
  const uint32_t u24 = a.u24_override ? a.u24_override[r] : philox_u24(a.seed[r], (uint64_t)a.step[r]);

  // ---- pass A: bins linear in (max - logit); bin 0 holds the largest logits
  // weights vanish beyond (max - l)/T > 27.73, so the bins cover 28 T logit units
  const float scale_a = (float)SMP_BINS / (28.f * temperature);
  for (int i = tid; i < SMP_BINS; i += SMP_THREADS) { sh.hist[i] = 0ull; sh.cnt[i] = 0u; }
  if (tid == 0) { sh.carried = 0ull; sh.kmin = 0xffffffffu; sh.kmax = 0u; }
  __syncthreads();
  unsigned long long mysum = 0ull;
  for (int i = tid; i < V; i += SMP_THREADS) {
    const float x = lg[i];
    const unsigned long long w = smp_weight(x, mx, inv_t_log2e);
    const int bin = min(SMP_BINS - 1, (int)((mx - x) * scale_a));
    atomicAdd(&sh.hist[bin], w);
    atomicAdd(&sh.cnt[bin], 1u);
    mysum += w;
  }
  unsigned long long total;
  block_excl_scan_u64(mysum, sh.wtot, &sh.total);
  total = sh.total;
  unsigned long long cut = __double2ull_rd((double)a.top_p[r] * (double)total);
  if (cut > total) cut = total;
  smp_select_bin(sh, cut);
  const int bin_a = sh.sel_bin;
  // key range of the selected bin
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
  // ---- passes B: exact refinement in key space until one key remains
  for (int pass = 0; pass < 4 && kmax > kmin; ++pass) {
    const unsigned long long width = (unsigned long long)(kmax - kmin) + 1ull;
    __syncthreads();
    for (int i = tid; i < SMP_BINS; i += SMP_THREADS) { sh.hist[i] = 0ull; sh.cnt[i] = 0u; }
    __syncthreads();
    for (int i = tid; i < V; i += SMP_THREADS) {
      const float x = lg[i];
      const uint32_t k = ordered_key(x);
      if (k >= kmin && k <= kmax) {
        const int j = (int)(((unsigned long long)(k - kmin) * SMP_BINS) / width);
        const int bin = SMP_BINS - 1 - j;            // descending key = ascending bin
        atomicAdd(&sh.hist[bin], smp_weight(x, mx, inv_t_log2e));
        atomicAdd(&sh.cnt[bin], 1u);
      }
    }
    __syncthreads();
    smp_select_bin(sh, cut);
    const unsigned long long j = (unsigned long long)(SMP_BINS - 1 - sh.sel_bin);
    // keys k with floor((k - kmin) * BINS / width) == j
    const unsigned long long lo = (j * width + SMP_BINS - 1) / SMP_BINS;
    const unsigned long long hi = ((j + 1) * width + SMP_BINS - 1) / SMP_BINS - 1;
    kmax = kmin + (uint32_t)hi;
    kmin = kmin + (uint32_t)lo;
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

  // ---- inverse CDF over nucleus members in ascending id order; thread = contiguous id range
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

// ---------------------------------------------------------------- decode bookkeeping
__global__ void prepare_rows_kernel(const uint8_t *active_mask, const int *in_use, const int *ctx_len,
                                    const int *pending, int B, int *row_token, int *row_pos, int *row_active,
                                    int *row_slot, int *do_sample) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= B) return;
  const int act = (active_mask[s] != 0 && in_use[s] != 0) ? 1 : 0;
  row_active[s] = act;
  row_slot[s] = s;
  row_pos[s] = act ? ctx_len[s] : 0;
  row_token[s] = act ? pending[s] : 0;
  do_sample[s] = act;
}

__global__ void advance_kernel(const int *row_active, const int *sampled, int B, int *ctx_len, int *step, int *pending,
                               int *out_tokens) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= B) return;
  if (row_active[s]) {
    const int tok = sampled[s];
    pending[s] = tok;
    ctx_len[s] += 1;
    step[s] += 1;
    out_tokens[s] = tok;
  } else {
    out_tokens[s] = -1;
  }
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
  __half *kp = base + ((size_t)g * KV_BLOCK + pos % KV_BLOCK) * kv.hd + i;
  __half *vp = kp + (size_t)kv.n_kv * KV_BLOCK * kv.hd;
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
  __half *kp = base + ((size_t)g * KV_BLOCK + t % KV_BLOCK) * kv.hd + i;
  *kp = __float2half_rn(rad * cospif(2.0f * u2));
  *(kp + (size_t)kv.n_kv * KV_BLOCK * kv.hd) = __float2half_rn(rad * sinpif(2.0f * u2));
}

template <int HD>
cudaError_t launch_attn_hd(int group, dim3 grid, cudaStream_t st, const float *q, const Rows &rows, int nq,
                           const KvLayout &kv, int layer, int max_splits, float *pa, float *pm) {
  switch (group) {
    case 1: attn_split_kernel<HD, 1><<<grid, ATT_THREADS, 0, st>>>(q, rows, nq, kv, layer, max_splits, pa, pm); break;
    case 2: attn_split_kernel<HD, 2><<<grid, ATT_THREADS, 0, st>>>(q, rows, nq, kv, layer, max_splits, pa, pm); break;
    case 4: attn_split_kernel<HD, 4><<<grid, ATT_THREADS, 0, st>>>(q, rows, nq, kv, layer, max_splits, pa, pm); break;
    case 8: attn_split_kernel<HD, 8><<<grid, ATT_THREADS, 0, st>>>(q, rows, nq, kv, layer, max_splits, pa, pm); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_resid_norm(float *h, int H, const __nv_bfloat16 *embed, const Rows &rows, const GemmOut *prev,
                              const __nv_bfloat16 *gains, float eps, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                              cudaStream_t st) {
  GemmOut g{};
  if (prev) g = *prev;
  resid_norm_kernel<<<rows.R, NORM_THREADS, 0, st>>>(h, H, embed, rows, g, prev ? 0 : 1, gains, eps, out_hi, out_lo);
  return cudaGetLastError();
}

cudaError_t launch_qkv_post(const GemmOut &qkv, const Rows &rows, const float2 *rope_tab, int nq, const KvLayout &kv,
                            int layer, float *q_out, cudaStream_t st) {
  qkv_post_kernel<<<rows.R, 256, 0, st>>>(qkv, rows, rope_tab, nq, kv, layer, q_out);
  return cudaGetLastError();
}

cudaError_t launch_attention(const float *q, const Rows &rows, int nq, const KvLayout &kv, int layer, int max_splits,
                             float *part_acc, float *part_ml, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo,
                             cudaStream_t st) {
  const dim3 grid(max_splits, kv.n_kv, rows.R);
  const int group = nq / kv.n_kv;
  cudaError_t e;
  if (kv.hd == 128) e = launch_attn_hd<128>(group, grid, st, q, rows, nq, kv, layer, max_splits, part_acc, part_ml);
  else if (kv.hd == 64) e = launch_attn_hd<64>(group, grid, st, q, rows, nq, kv, layer, max_splits, part_acc, part_ml);
  else return cudaErrorInvalidValue;
  if (e != cudaSuccess) return e;
  attn_combine_kernel<<<rows.R, 256, 0, st>>>(rows, nq, kv.hd, max_splits, part_acc, part_ml, out_hi, out_lo);
  return cudaGetLastError();
}

cudaError_t launch_swiglu(const GemmOut &gu, int R, int F, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, cudaStream_t st) {
  swiglu_kernel<<<dim3((F + 255) / 256, R), 256, 0, st>>>(gu, F, out_hi, out_lo);
  return cudaGetLastError();
}

cudaError_t launch_split(const float *x, int R, int K, __nv_bfloat16 *hi, __nv_bfloat16 *lo, cudaStream_t st) {
  const size_t n = (size_t)R * K;
  split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(x, n, hi, lo);
  return cudaGetLastError();
}

cudaError_t launch_sampler(const SampleArgs &a, int R, cudaStream_t st) {
  sampler_kernel<<<R, SMP_THREADS, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_prepare_rows(const uint8_t *active_mask, const int *in_use, const int *ctx_len, const int *pending,
                                int B, int *row_token, int *row_pos, int *row_active, int *row_slot, int *do_sample,
                                cudaStream_t st) {
  prepare_rows_kernel<<<(B + 127) / 128, 128, 0, st>>>(active_mask, in_use, ctx_len, pending, B, row_token, row_pos,
                                                       row_active, row_slot, do_sample);
  return cudaGetLastError();
}

cudaError_t launch_advance(const int *row_active, const int *sampled, int B, int *ctx_len, int *step, int *pending,
                           int *out_tokens, cudaStream_t st) {
  advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(row_active, sampled, B, ctx_len, step, pending, out_tokens);
  return cudaGetLastError();
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
