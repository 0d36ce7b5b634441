// Token-wise kernels of a multi-head latent attention (MLA) layer around the attention kernel: cache append with
// the latent's RMSNorm and the rotary key's rotation, the query's parts, the value part of the up-projection,
// and the set-up / debug helpers of the latent pool.  Every reduction has one fixed order.
#include "mla.cuh"

#include "checks.cuh"
#include "launch.cuh"
#include "ptx.cuh"

namespace corun {

namespace {

__device__ __forceinline__ void mla_split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

constexpr int MLA_POST_THREADS = 256;

__device__ __forceinline__ void mla_store_split4(float4 y, __nv_bfloat16 *hi, __nv_bfloat16 *lo) {
  __nv_bfloat16 a[4], b[4];
  mla_split_bf16(y.x, a[0], b[0]);
  mla_split_bf16(y.y, a[1], b[1]);
  mla_split_bf16(y.z, a[2], b[2]);
  mla_split_bf16(y.w, a[3], b[3]);
  *reinterpret_cast<uint2 *>(hi) = *reinterpret_cast<const uint2 *>(a);
  *reinterpret_cast<uint2 *>(lo) = *reinterpret_cast<const uint2 *>(b);
}
// (a, b) pairs of four consecutive rotation indices -> rotated (a', b'); t: (cos, sin) of those indices
__device__ __forceinline__ void mla_rotate4(const float4 a, const float4 b, const float2 *t, float4 &ra, float4 &rb) {
  const float4 t01 = *reinterpret_cast<const float4 *>(t), t23 = *reinterpret_cast<const float4 *>(t + 2);
  ra = make_float4(a.x * t01.x - b.x * t01.y, a.y * t01.z - b.y * t01.w, a.z * t23.x - b.z * t23.y, a.w * t23.z - b.w * t23.w);
  rb = make_float4(a.x * t01.y + b.x * t01.x, a.y * t01.w + b.y * t01.z, a.z * t23.y + b.z * t23.x, a.w * t23.w + b.w * t23.z);
}

// One CTA per row; four consecutive columns per thread and pass (nope, rope / 2 and rank are multiples of 4).
__global__ void __launch_bounds__(MLA_POST_THREADS)
mla_post_kernel(GemmOut qkv, Rows rows, const float2 *__restrict__ rope_tab, MlaDims d, const __nv_bfloat16 *__restrict__ gains,
                float eps, MlaCache cache, int rows_per_head, __nv_bfloat16 *__restrict__ qn_hi, __nv_bfloat16 *__restrict__ qn_lo,
                float *__restrict__ q_rope, int *status) {
  griddep_launch_dependents();
  griddep_wait();
  __shared__ float scratch[MLA_POST_THREADS / 32];
  const int r = blockIdx.x, tid = threadIdx.x;
  if (rows.active[r] == 0) return;                   // a padding row: no cache write, its query is never used
  const int pos = rows.pos[r];
  const int qw = d.nope + d.rope, QD = d.nh * qw, half = d.rope >> 1;
  const float2 *tab = rope_tab + (size_t)pos * half;   // (cos, sin) of the row's position
#ifdef CORUN_CHECKED
  if (!check_slot_pos(rows.slot[r], cache.n_slots, pos, cache.max_blocks, KV_BLOCK)) {
    if (tid == 0) atomicCAS(status, 0, DEV_BAD_INDEX);
    return;
  }
#endif
  const int blk = cache.block_table[(size_t)rows.slot[r] * cache.max_blocks + pos / KV_BLOCK];
#ifdef CORUN_CHECKED
  if (!check_page(blk, cache.pool_blocks)) {
    if (tid == 0) atomicCAS(status, 0, DEV_BAD_INDEX);
    return;
  }
#endif
  const int row_halfs = d.rank + d.rope, off = pos % KV_BLOCK;   // the row's cache position: mla_cache_at(.., blk, off, e)
  // the latent's values are requested first and used last: the sums of the GEMM's partials behind every load
  // below overlap instead of queueing behind the block-wide reduction
  float4 x = make_float4(0.f, 0.f, 0.f, 0.f);        // rank <= 4 * threads
  if (4 * tid < d.rank) x = gemm_load4(qkv, r, QD + 4 * tid);
  // ---- the query: no-rope parts as bf16 hi/lo (head-major), rotary parts rotated, fp32
  for (int i = 4 * tid; i < d.nh * d.nope; i += 4 * MLA_POST_THREADS) {
    const int h = i / d.nope, j = i - h * d.nope;
    const size_t o = ((size_t)h * rows_per_head + r) * d.nope + j;
    mla_store_split4(gemm_load4(qkv, r, h * qw + j), qn_hi + o, qn_lo + o);
  }
  for (int i = 4 * tid; i < d.nh * half; i += 4 * MLA_POST_THREADS) {
    const int h = i / half, j = i - h * half;
    float4 ra, rb;
    mla_rotate4(gemm_load4(qkv, r, h * qw + d.nope + j), gemm_load4(qkv, r, h * qw + d.nope + j + half), tab + j, ra, rb);
    float *q = q_rope + ((size_t)r * d.nh + h) * d.rope + j;
    *reinterpret_cast<float4 *>(q) = ra;
    *reinterpret_cast<float4 *>(q + half) = rb;
  }
  // ---- the cache row: rotated rotary key; RMSNorm of the latent (sum of squares: thread-serial ascending, xor
  //      butterfly in the warp, warp totals ascending)
  if (4 * tid < half) {
    const int j = 4 * tid;
    float4 ra, rb;
    mla_rotate4(gemm_load4(qkv, r, QD + d.rank + j), gemm_load4(qkv, r, QD + d.rank + j + half), tab + j, ra, rb);
    __half2 oa[2] = {__floats2half2_rn(ra.x, ra.y), __floats2half2_rn(ra.z, ra.w)};
    __half2 ob[2] = {__floats2half2_rn(rb.x, rb.y), __floats2half2_rn(rb.z, rb.w)};
    *reinterpret_cast<uint2 *>(mla_cache_at(cache, row_halfs, blk, off, d.rank + j)) = *reinterpret_cast<const uint2 *>(oa);
    *reinterpret_cast<uint2 *>(mla_cache_at(cache, row_halfs, blk, off, d.rank + j + half)) = *reinterpret_cast<const uint2 *>(ob);
  }
  float ss = 0.f;
  ss = fmaf(x.x, x.x, ss); ss = fmaf(x.y, x.y, ss); ss = fmaf(x.z, x.z, ss); ss = fmaf(x.w, x.w, ss);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((tid & 31) == 0) scratch[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < MLA_POST_THREADS / 32; ++w) tot += scratch[w];
  const float inv = rsqrtf(tot / (float)d.rank + eps);
  if (4 * tid < d.rank) {
    const uint2 raw = *reinterpret_cast<const uint2 *>(gains + 4 * tid);
    const __nv_bfloat162 *g2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
    const float2 ga = __bfloat1622float2(g2[0]), gb = __bfloat1622float2(g2[1]);
    __half2 o[2] = {__floats2half2_rn(x.x * inv * ga.x, x.y * inv * ga.y), __floats2half2_rn(x.z * inv * gb.x, x.w * inv * gb.y)};
    *reinterpret_cast<uint2 *>(mla_cache_at(cache, row_halfs, blk, off, 4 * tid)) = *reinterpret_cast<const uint2 *>(o);
  }
}

__global__ void __launch_bounds__(256)
mla_ao_split_kernel(const float *__restrict__ uv, int R, int rows_per_head, MlaDims d, __nv_bfloat16 *__restrict__ ao_hi,
                    __nv_bfloat16 *__restrict__ ao_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int r = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= d.nh * d.vh) return;
  const int h = i / d.vh, j = i - h * d.vh;
  __nv_bfloat16 a, b;
  mla_split_bf16(uv[((size_t)h * rows_per_head + r) * (d.nope + d.vh) + d.nope + j], a, b);
  ao_hi[(size_t)r * d.nh * d.vh + i] = a;
  ao_lo[(size_t)r * d.nh * d.vh + i] = b;
}

__global__ void mla_transpose_uk_kernel(const __nv_bfloat16 *__restrict__ wkv_b, MlaDims d, __nv_bfloat16 *__restrict__ out) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t n = (size_t)d.nh * d.rank * d.nope;
  if (idx >= n) return;
  const int i = (int)(idx % d.nope);
  const int c = (int)((idx / d.nope) % d.rank);
  const int h = (int)(idx / ((size_t)d.nope * d.rank));
  out[idx] = wkv_b[((size_t)h * (d.nope + d.vh) + i) * d.rank + c];
}

__device__ __forceinline__ uint64_t mla_mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Synthetic cache contents for timing runs: position-hashed normals, one thread per pair of values.
__global__ void mla_fill_kernel(MlaCache cache, int row_halfs, int layer, int slot, int n, float std, uint64_t seed) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int pairs = row_halfs / 2;
  if (idx >= (size_t)n * pairs) return;
  const int t = (int)(idx / pairs), e = (int)(idx - (size_t)t * pairs);
  const uint64_t h = mla_mix64(seed ^ mla_mix64(((uint64_t)slot << 48) ^ ((uint64_t)layer << 40) ^ ((uint64_t)t << 16) ^ (uint64_t)e));
  const float u1 = ((float)(uint32_t)(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
  const float u2 = (float)(uint32_t)((h >> 8) & 0xFFFFFFu) * (1.0f / 16777216.0f);
  const float rad = sqrtf(-2.0f * logf(u1)) * std;
  const int blk = cache.block_table[(size_t)slot * cache.max_blocks + t / KV_BLOCK];
  __half *row = mla_cache_at(cache, row_halfs, blk, t % KV_BLOCK, 2 * e);   // a pair never straddles a block of 64 dims
  row[0] = __float2half_rn(rad * cospif(2.0f * u2));
  row[1] = __float2half_rn(rad * sinpif(2.0f * u2));
}

__global__ void mla_copy_kernel(MlaCache cache, int row_halfs, int slot, int pos0, int n, float *buf, int write) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)n * row_halfs) return;
  const int t = pos0 + (int)(idx / row_halfs), e = (int)(idx % row_halfs);
  const int blk = cache.block_table[(size_t)slot * cache.max_blocks + t / KV_BLOCK];
  __half *p = mla_cache_at(cache, row_halfs, blk, t % KV_BLOCK, e);
  if (write) *p = __float2half_rn(buf[idx]);
  else buf[idx] = __half2float(*p);
}

}  // namespace

cudaError_t launch_mla_post(const GemmOut &qkv, const Rows &rows, const float2 *rope_tab, const MlaDims &d,
                            const __nv_bfloat16 *kv_gains, float eps, const MlaCache &cache, int rows_per_head,
                            __nv_bfloat16 *qn_hi, __nv_bfloat16 *qn_lo, float *q_rope, int *d_status, cudaStream_t st) {
  return launch_k(mla_post_kernel, dim3(rows.R), dim3(MLA_POST_THREADS), 0, st, true, qkv, rows, rope_tab, d, kv_gains, eps, cache,
                  rows_per_head, qn_hi, qn_lo, q_rope, d_status);
}

cudaError_t launch_mla_ao_split(const float *uv, int R, int rows_per_head, const MlaDims &d, __nv_bfloat16 *ao_hi,
                                __nv_bfloat16 *ao_lo, cudaStream_t st) {
  return launch_k(mla_ao_split_kernel, dim3((d.nh * d.vh + 255) / 256, R), dim3(256), 0, st, true, uv, R, rows_per_head, d, ao_hi, ao_lo);
}

cudaError_t launch_mla_transpose_uk(const __nv_bfloat16 *wkv_b, const MlaDims &d, __nv_bfloat16 *out, cudaStream_t st) {
  const size_t n = (size_t)d.nh * d.rank * d.nope;
  mla_transpose_uk_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(wkv_b, d, out);
  return cudaGetLastError();
}

cudaError_t launch_mla_fill(const MlaCache &cache, int row_halfs, int layer, int slot, int n, float std, uint64_t seed, cudaStream_t st) {
  const size_t tot = (size_t)n * (row_halfs / 2);
  if (tot == 0) return cudaSuccess;
  mla_fill_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(cache, row_halfs, layer, slot, n, std, seed);
  return cudaGetLastError();
}

cudaError_t launch_mla_copy(const MlaCache &cache, int row_halfs, int slot, int pos0, int n, float *buf, int write, cudaStream_t st) {
  const size_t tot = (size_t)n * row_halfs;
  if (tot == 0) return cudaSuccess;
  mla_copy_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(cache, row_halfs, slot, pos0, n, buf, write);
  return cudaGetLastError();
}

}  // namespace corun
