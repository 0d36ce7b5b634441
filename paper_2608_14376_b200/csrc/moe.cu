// Mixture-of-Experts feed-forward block without groups: two plain decode GEMMs over all experts with a
// masked, probability-weighted SwiGLU between them (see include/corun_moe.h for the formulation and why
// it is position-invariant).  The kernels here are the router's softmax / top-k, the masked SwiGLU and
// the read-out of the second GEMM; the GEMMs are gemm.cu's.
#include <cuda_bf16.h>
#include <math_constants.h>

#include <new>
#include <vector>

#include "../../include/corun_moe.h"
#include "gemm.cuh"
#include "launch.cuh"
#include "moe.cuh"
#include "ops.cuh"
#include "ptx.cuh"

using namespace corun;

namespace {

using bf16 = __nv_bfloat16;
constexpr int MOE_MAX_TOPK = 16;
constexpr int MOE_MAX_EXPERTS = 256;

#define MCK(call)                               \
  do {                                          \
    cudaError_t ce_ = (call);                   \
    if (ce_ != cudaSuccess) {                   \
      g_last_cuda_error = (int)ce_;             \
      return CORUN_ECUDA;                       \
    }                                           \
  } while (0)

__device__ __forceinline__ void moe_split(float x, bf16 &hi, bf16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// One warp routes one row: softmax over the E router logits (load(e) gives logit e), then top_k by repeated arg-max
// with ties to the lower id.  Lane l holds experts l, l + 32, ...; the sum of the exponentials is each lane's
// experts in ascending id, then a fixed butterfly over the lanes.  Writes the routing and the row of SwiGLU weights
// w[r, 0 .. E + S): p_e for the selected experts, 0 for the others, 1 for the shared ones.
template <typename LoadLogit>
__device__ __forceinline__ void moe_route_row(LoadLogit load, int r, int lane, int E, int S, int top_k, int renormalize,
                                              float *__restrict__ w, int *__restrict__ experts, float *__restrict__ probs) {
  constexpr int PER = MOE_MAX_EXPERTS / 32;
  float z[PER];
  float mx = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int e = lane + 32 * j;
    z[j] = e < E ? load(e) : -CUDART_INF_F;
    mx = fmaxf(mx, z[j]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int e = lane + 32 * j;
    z[j] = e < E ? expf(z[j] - mx) : -1.f;           // -1: not an expert
    if (e < E) sum += z[j];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  float *wr = w + (size_t)r * (E + S);
  for (int e = lane; e < E; e += 32) wr[e] = 0.f;
  for (int s = lane; s < S; s += 32) wr[E + s] = 1.f;
  __syncwarp();
  int ids[MOE_MAX_TOPK];
  float ps[MOE_MAX_TOPK];
  float picked = 0.f;                                // sum of the selected probabilities, in selection order
  for (int k = 0; k < top_k; ++k) {
    float bz = -1.f;                                 // this lane's best: largest value, lowest id on ties
    int be = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < PER; ++j)
      if (z[j] > bz) { bz = z[j]; be = lane + 32 * j; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float oz = __shfl_xor_sync(0xffffffffu, bz, o);
      const int oe = __shfl_xor_sync(0xffffffffu, be, o);
      if (oz > bz || (oz == bz && oe < be)) { bz = oz; be = oe; }
    }
    if (be >= E) be = k;                             // a row of NaNs: any valid id
    const float p = __fdiv_rn(bz, sum);
#pragma unroll
    for (int j = 0; j < PER; ++j)
      if (lane + 32 * j == be) z[j] = -2.f;          // taken
    ids[k] = be;
    ps[k] = p;
    picked += p;
  }
  if (lane == 0)
    for (int k = 0; k < top_k; ++k) {
      const float p = renormalize ? __fdiv_rn(ps[k], picked) : ps[k];
      wr[ids[k]] = p;
      if (experts) experts[(size_t)r * top_k + k] = ids[k];
      if (probs) probs[(size_t)r * top_k + k] = p;
    }
}

// Router of one row per CTA: logits = Wr x on the CUDA cores (E dot products of H terms: far too little for a
// tensor-core launch of its own), then the routing above.  x is the row's bf16 hi + lo pair (exactly what the
// GEMMs of the block see); every warp takes experts warp, warp + 32, ...: a lane adds its terms in ascending
// order (8 consecutive terms per step, the weights of four steps requested together), then a fixed butterfly
// over the lanes.  A row's routing depends on the row alone.
constexpr int ROUTER_THREADS = 1024;
__global__ void __launch_bounds__(ROUTER_THREADS) moe_router_kernel(const bf16 *__restrict__ x_hi, const bf16 *__restrict__ x_lo, int H,
                                                                    const bf16 *__restrict__ Wr, int E, int S, int top_k,
                                                                    int renormalize, float *__restrict__ w,
                                                                    int *__restrict__ experts, float *__restrict__ probs) {
  griddep_launch_dependents();
  extern __shared__ float xs[];                      // the row as fp32 [H]
  __shared__ float logit[MOE_MAX_EXPERTS];
  const int r = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  griddep_wait();
  for (int i = 4 * tid; i < H; i += 4 * ROUTER_THREADS) {
    const uint2 rh = *reinterpret_cast<const uint2 *>(x_hi + (size_t)r * H + i), rl = *reinterpret_cast<const uint2 *>(x_lo + (size_t)r * H + i);
    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&rh), *l2 = reinterpret_cast<const __nv_bfloat162 *>(&rl);
    const float2 h0 = __bfloat1622float2(h2[0]), h1 = __bfloat1622float2(h2[1]), l0 = __bfloat1622float2(l2[0]), l1 = __bfloat1622float2(l2[1]);
    *reinterpret_cast<float4 *>(xs + i) = make_float4(h0.x + l0.x, h0.y + l0.y, h1.x + l1.x, h1.y + l1.y);
  }
  __syncthreads();
  for (int e = warp; e < E; e += ROUTER_THREADS / 32) {
    const bf16 *wrow = Wr + (size_t)e * H;
    float acc = 0.f;
    for (int i0 = 8 * lane; i0 < H; i0 += 4 * 8 * 32) {
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 8 * 32;
        raw[u] = i < H ? __ldg(reinterpret_cast<const uint4 *>(wrow + i)) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 8 * 32;
        if (i >= H) break;
        const __nv_bfloat162 *w2 = reinterpret_cast<const __nv_bfloat162 *>(&raw[u]);
        const float4 xa = *reinterpret_cast<const float4 *>(xs + i), xb = *reinterpret_cast<const float4 *>(xs + i + 4);
        const float2 w0 = __bfloat1622float2(w2[0]), w1 = __bfloat1622float2(w2[1]), w2f = __bfloat1622float2(w2[2]), w3 = __bfloat1622float2(w2[3]);
        acc = fmaf(w0.x, xa.x, acc); acc = fmaf(w0.y, xa.y, acc); acc = fmaf(w1.x, xa.z, acc); acc = fmaf(w1.y, xa.w, acc);
        acc = fmaf(w2f.x, xb.x, acc); acc = fmaf(w2f.y, xb.y, acc); acc = fmaf(w3.x, xb.z, acc); acc = fmaf(w3.y, xb.w, acc);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) logit[e] = acc;
  }
  __syncthreads();
  if (warp == 0) moe_route_row([&](int e) { return logit[e]; }, r, lane, E, S, top_k, renormalize, w, experts, probs);
}

// h[r, e*F + f] = w[r, e] * silu(gate) * up as a bf16 hi/lo pair; zeros where w[r, e] == 0 (nothing is read
// there).  gate = GEMM-1 column e*2F + f, up = column e*2F + F + f.  Four f per thread.
__global__ void __launch_bounds__(256) moe_swiglu_kernel(GemmOut gu, const float *__restrict__ w, int F, int n_blocks,
                                                         bf16 *__restrict__ out_hi, bf16 *__restrict__ out_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int r = blockIdx.y;
  const int per_block = F / 4;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= per_block * n_blocks) return;
  const int e = idx / per_block, f = (idx - e * per_block) * 4;
  const float we = w[(size_t)r * n_blocks + e];
  float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
  if (we != 0.f) {
    const float4 g = gemm_load4(gu, r, e * 2 * F + f), u = gemm_load4(gu, r, e * 2 * F + F + f);
    y = make_float4(we * (g.x / (1.f + expf(-g.x)) * u.x), we * (g.y / (1.f + expf(-g.y)) * u.y),
                    we * (g.z / (1.f + expf(-g.z)) * u.z), we * (g.w / (1.f + expf(-g.w)) * u.w));
  }
  bf16 a[4], b[4];
  moe_split(y.x, a[0], b[0]);
  moe_split(y.y, a[1], b[1]);
  moe_split(y.z, a[2], b[2]);
  moe_split(y.w, a[3], b[3]);
  const size_t o = (size_t)r * n_blocks * F + (size_t)e * F + f;
  *reinterpret_cast<uint2 *>(out_hi + o) = *reinterpret_cast<const uint2 *>(a);
  *reinterpret_cast<uint2 *>(out_lo + o) = *reinterpret_cast<const uint2 *>(b);
}

// y[r, :] = the second GEMM's result (partials of a tile added in ascending CTA order).
__global__ void __launch_bounds__(256) moe_readout_kernel(GemmOut d, int H, float *__restrict__ y) {
  griddep_launch_dependents();
  griddep_wait();
  const int r = blockIdx.y;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= H) return;
  *reinterpret_cast<float4 *>(y + (size_t)r * H + i) = gemm_load4(d, r, i);
}

// ---------------------------------------------------------------- grouped form
// One CTA per expert (routed experts, then the shared ones).  Every CTA counts the rows of ALL experts (the table
// w[r, e] != 0 is small and comes from L2), so that it knows where its own expert's groups begin (experts ascending,
// 64 rows per group) without a second kernel; it then writes its groups' table entries and hands its rows, in
// ascending row order, consecutive slots (slot_of is expert-major: [E + S][R]).  CTA 0 also clears the entries of
// the groups nobody needs and publishes the number of groups in use.
constexpr int MOE_GROUP_THREADS = 512;
__global__ void __launch_bounds__(MOE_GROUP_THREADS) moe_group_kernel(const float *__restrict__ w, const int *__restrict__ active, int R,
                                                       int NB, int E, int F, MoeGroups g) {
  griddep_launch_dependents();
  __shared__ int cnt[MOE_MAX_EXPERTS + 8];
  __shared__ float wsel[256];                        // the own expert's weight per row, 0 = not selected
  __shared__ unsigned char act[256];
  __shared__ int first_s, total_s;
  const int e = (int)blockIdx.x, tid = (int)threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < NB; i += MOE_GROUP_THREADS) cnt[i] = 0;
  griddep_wait();
  w = after_wait(w); active = after_wait(active);    // no load through them may move up across the wait
  for (int r = tid; r < R; r += MOE_GROUP_THREADS) { act[r] = active[r] != 0; wsel[r] = 0.f; }
  __syncthreads();
  {
    // sixteen independent loads per thread in flight
    const int total = R * NB;
    for (int i0 = tid; i0 < total; i0 += MOE_GROUP_THREADS * 16) {
      float v[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) v[k] = i0 + MOE_GROUP_THREADS * k < total ? w[i0 + MOE_GROUP_THREADS * k] : 0.f;
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int i = i0 + MOE_GROUP_THREADS * k;
        if (i < total && v[k] != 0.f) {
          const int r = i / NB, ee = i - r * NB;
          if (act[r]) {
            atomicAdd(&cnt[ee], 1);                  // integer counts: the order of the additions does not matter
            if (ee == e) wsel[r] = v[k];
          }
        }
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    // groups before this expert, and in all: lanes take experts lane, lane + 32, ...
    int before = 0, all = 0;
    for (int ee = lane; ee < NB; ee += 32) {
      const int n = (cnt[ee] + MOE_GROUP_ROWS - 1) / MOE_GROUP_ROWS;
      all += n;
      if (ee < e) before += n;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      before += __shfl_xor_sync(0xffffffffu, before, o);
      all += __shfl_xor_sync(0xffffffffu, all, o);
    }
    if (lane == 0) { first_s = before; total_s = all < g.n_groups_max ? all : g.n_groups_max; }
  }
  __syncthreads();
  const int first = first_s, used = total_s;
  if (e == 0) {
    for (int u = used + tid; u < g.n_groups_max; u += MOE_GROUP_THREADS) {   // groups nobody needs
      g.tab_up[3 * u] = 0; g.tab_up[3 * u + 1] = 0; g.tab_up[3 * u + 2] = 0;
      g.tab_down[3 * u] = 0; g.tab_down[3 * u + 1] = 0; g.tab_down[3 * u + 2] = 0;
      g.group_expert[u] = -1;
    }
    if (tid == 0) g.tab_up[3 * g.n_groups_max] = g.tab_down[3 * g.n_groups_max] = used;   // what the GEMMs walk
  }
  const int n_groups = (cnt[e] + MOE_GROUP_ROWS - 1) / MOE_GROUP_ROWS;
  for (int k = tid; k < n_groups; k += MOE_GROUP_THREADS) {
    const int u = first + k;
    if (u >= g.n_groups_max) break;                 // cannot happen: n_groups_max bounds the sum
    const int rows = min(MOE_GROUP_ROWS, cnt[e] - k * MOE_GROUP_ROWS);
    g.tab_up[3 * u] = e * 2 * F; g.tab_up[3 * u + 1] = 0; g.tab_up[3 * u + 2] = rows;
    g.tab_down[3 * u] = 0; g.tab_down[3 * u + 1] = e * F / GEMM_BLOCK_K; g.tab_down[3 * u + 2] = rows;
    g.group_expert[u] = e;
  }
  if (warp == 0) {
    int base = first * MOE_GROUP_ROWS;               // slot of the expert's next row
    for (int r0 = 0; r0 < R; r0 += 32) {
      const int r = r0 + lane;
      const float wv = r < R ? wsel[r] : 0.f;
      const bool on = wv != 0.f;
      const unsigned m = __ballot_sync(0xffffffffu, on);
      int slot = -1;
      if (on) {
        slot = base + __popc(m & ((1u << lane) - 1u));
        g.slot_row[slot] = r;
        g.slot_w[slot] = wv;
      }
      if (r < R) g.slot_of[(size_t)e * R + r] = slot;
      base += __popc(m);
    }
  }
}

// The gathered activation rows: one warp per slot of the groups in use (all of a row's loads requested before the
// first store).  H % 256 == 0 up to 4096, else eight 16-byte pieces per lane at a time.
__global__ void __launch_bounds__(256) moe_gather_kernel(const bf16 *__restrict__ x_hi, const bf16 *__restrict__ x_lo, int H,
                                                         MoeGroups g, bf16 *__restrict__ xg_hi, bf16 *__restrict__ xg_lo) {
  griddep_launch_dependents();
  griddep_wait();
  x_hi = after_wait(x_hi); x_lo = after_wait(x_lo);
  const int lane = threadIdx.x & 31;
  const int n_slots = g.tab_up[3 * g.n_groups_max] * MOE_GROUP_ROWS;
  const int n_warps = (int)(gridDim.x * (blockDim.x >> 5));
  for (int slot = (int)(blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)); slot < n_slots; slot += n_warps) {
    if (slot % MOE_GROUP_ROWS >= g.tab_up[3 * (slot / MOE_GROUP_ROWS) + 2]) continue;   // no row in this slot
    const int r = g.slot_row[slot];
    const uint4 *sh = reinterpret_cast<const uint4 *>(x_hi + (size_t)r * H), *sl = reinterpret_cast<const uint4 *>(x_lo + (size_t)r * H);
    uint4 *dh = reinterpret_cast<uint4 *>(xg_hi + (size_t)slot * H), *dl = reinterpret_cast<uint4 *>(xg_lo + (size_t)slot * H);
    for (int i0 = lane; i0 < H / 8; i0 += 32 * 8) {
      uint4 a[8], b[8];
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (i0 + 32 * k < H / 8) { a[k] = sh[i0 + 32 * k]; b[k] = sl[i0 + 32 * k]; }
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (i0 + 32 * k < H / 8) { dh[i0 + 32 * k] = a[k]; dl[i0 + 32 * k] = b[k]; }
    }
  }
}

__global__ void __launch_bounds__(256) moe_swiglu_grouped_kernel(const float *__restrict__ gu, const float *__restrict__ w,
                                                                 int NB, int F, MoeGroups g, bf16 *__restrict__ hg_hi,
                                                                 bf16 *__restrict__ hg_lo) {
  griddep_launch_dependents();
  griddep_wait();
  const int slot = blockIdx.x;
  if (slot % MOE_GROUP_ROWS >= g.tab_up[3 * (slot / MOE_GROUP_ROWS) + 2]) return;   // no row in this slot
  const int r = g.slot_row[slot];
  const int e = g.group_expert[slot / MOE_GROUP_ROWS];
  const float we = w[(size_t)r * NB + e];
  const float *row = gu + (size_t)slot * 2 * F;
  for (int f = threadIdx.x * 4; f < F; f += blockDim.x * 4) {
    const float4 a = *reinterpret_cast<const float4 *>(row + f), u = *reinterpret_cast<const float4 *>(row + F + f);
    const float4 y = make_float4(we * (a.x / (1.f + expf(-a.x)) * u.x), we * (a.y / (1.f + expf(-a.y)) * u.y),
                                 we * (a.z / (1.f + expf(-a.z)) * u.z), we * (a.w / (1.f + expf(-a.w)) * u.w));
    bf16 p[4], q[4];
    moe_split(y.x, p[0], q[0]);
    moe_split(y.y, p[1], q[1]);
    moe_split(y.z, p[2], q[2]);
    moe_split(y.w, p[3], q[3]);
    *reinterpret_cast<uint2 *>(hg_hi + (size_t)slot * F + f) = *reinterpret_cast<const uint2 *>(p);
    *reinterpret_cast<uint2 *>(hg_lo + (size_t)slot * F + f) = *reinterpret_cast<const uint2 *>(q);
  }
}

__global__ void __launch_bounds__(256) moe_combine_kernel(const float *__restrict__ yg, const int *__restrict__ active, int NB,
                                                          int H, MoeGroups g, float *__restrict__ y) {
  griddep_launch_dependents();
  griddep_wait();
  yg = after_wait(yg); active = after_wait(active);
  const int r = blockIdx.y;
  if (!active[r]) return;
  __shared__ int slots[MOE_MAX_EXPERTS + 8];         // the row's slots, experts ascending (shared experts last), compacted
  __shared__ int n_sel;
  if (threadIdx.x < 32) {
    int n = 0;
    for (int e0 = 0; e0 < NB; e0 += 32) {
      const int e = e0 + (int)threadIdx.x;
      const int slot = e < NB ? g.slot_of[(size_t)e * gridDim.y + r] : -1;
      const unsigned m = __ballot_sync(0xffffffffu, slot >= 0);
      if (slot >= 0) slots[n + __popc(m & ((1u << threadIdx.x) - 1u))] = slot;
      n += __popc(m);
    }
    if (threadIdx.x == 0) n_sel = n;
  }
  __syncthreads();
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= H) return;
  const int n = n_sel;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k0 = 0; k0 < n; k0 += 8) {                // eight loads in flight; the additions stay in ascending order
    float4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (k0 + k < n) v[k] = *reinterpret_cast<const float4 *>(yg + (size_t)slots[k0 + k] * H + i);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (k0 + k < n) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
  }
  *reinterpret_cast<float4 *>(y + (size_t)r * H + i) = acc;
}

}  // namespace

namespace corun {

cudaError_t launch_moe_group(const float *w, const int *active, int R, int E, int S, int F, const MoeGroups &g,
                             cudaStream_t st) {
  if (E + S > MOE_MAX_EXPERTS + 8 || F % GEMM_BLOCK_K || R > 256) return cudaErrorInvalidValue;
  return launch_k(moe_group_kernel, dim3(E + S), dim3(MOE_GROUP_THREADS), 0, st, true, w, active, R, E + S, E, F, g);
}

cudaError_t launch_moe_gather(const __nv_bfloat16 *x_hi, const __nv_bfloat16 *x_lo, int H, const MoeGroups &g,
                              __nv_bfloat16 *xg_hi, __nv_bfloat16 *xg_lo, cudaStream_t st) {
  const int blocks = (g.n_groups_max * MOE_GROUP_ROWS + 7) / 8;   // a warp per slot, as far as 1184 CTAs go
  return launch_k(moe_gather_kernel, dim3(blocks < 1184 ? blocks : 1184), dim3(256), 0, st, true, x_hi, x_lo, H, g, xg_hi, xg_lo);
}

cudaError_t launch_moe_swiglu_grouped(const float *gu, const float *w, int n_blocks, int F, const MoeGroups &g,
                                      __nv_bfloat16 *hg_hi, __nv_bfloat16 *hg_lo, cudaStream_t st) {
  return launch_k(moe_swiglu_grouped_kernel, dim3(g.n_groups_max * MOE_GROUP_ROWS), dim3(192), 0, st, true, gu, w, n_blocks, F, g,
                  hg_hi, hg_lo);
}

cudaError_t launch_moe_combine(const float *yg, const int *active, int R, int n_blocks, int H, const MoeGroups &g, float *y,
                               cudaStream_t st) {
  return launch_k(moe_combine_kernel, dim3((H / 4 + 255) / 256, R), dim3(256), 0, st, true, yg, active, n_blocks, H, g, y);
}

cudaError_t launch_moe_router(const bf16 *x_hi, const bf16 *x_lo, int H, const bf16 *Wr, int R, int E, int S, int top_k,
                              int renormalize, float *w, int *experts, float *probs, cudaStream_t st) {
  return launch_k(moe_router_kernel, dim3(R), dim3(ROUTER_THREADS), (size_t)H * sizeof(float), st, true, x_hi, x_lo, H, Wr, E, S, top_k,
                  renormalize, w, experts, probs);
}

cudaError_t launch_moe_swiglu(const GemmOut &gu, const float *w, int R, int F, int n_blocks, __nv_bfloat16 *out_hi,
                              __nv_bfloat16 *out_lo, cudaStream_t st) {
  return launch_k(moe_swiglu_kernel, dim3((n_blocks * (F / 4) + 255) / 256, R), dim3(256), 0, st, true, gu, w, F, n_blocks,
                  out_hi, out_lo);
}

}  // namespace corun

struct corun_moe {
  corun_moe_shape sh{};
  int B = 0, BN = 0, num_sms = 0;
  cudaStream_t st = nullptr;
  std::vector<void *> allocs;
  const bf16 *router = nullptr;                     // [E, H], borrowed
  bf16 *x_hi = nullptr, *x_lo = nullptr, *h_hi = nullptr, *h_lo = nullptr;
  float *out_gu = nullptr, *out_d = nullptr, *ws = nullptr, *w = nullptr;
  int *d_status = nullptr;
  GemmPlan p_gu, p_d;
  // grouped form (more than 64 padded rows): an expert's rows gathered into blocks of 64
  bool grouped = false;
  MoeGroups grp{};
  bf16 *xg_hi = nullptr, *xg_lo = nullptr, *hg_hi = nullptr, *hg_lo = nullptr;
  float *yg = nullptr;
  int *d_active = nullptr;
  GemmPlan p_gug, p_dng;
  int64_t weight_bytes = 0;
};

namespace {

template <typename T>
int moe_alloc(corun_moe *m, T **p, size_t n) {
  void *q = nullptr;
  if (cudaMalloc(&q, n * sizeof(T)) != cudaSuccess) return CORUN_ENOMEM;
  m->allocs.push_back(q);
  if (cudaMemset(q, 0, n * sizeof(T)) != cudaSuccess) return CORUN_ECUDA;
  *p = (T *)q;
  return CORUN_OK;
}

}  // namespace

extern "C" {

int corun_moe_create(const corun_moe_shape *shape, const void *router, const void *gate_up, const void *down,
                     int32_t B, void *cuda_stream, corun_moe **out) {
  if (!shape || !router || !gate_up || !down || !out || B < 1 || B > 256) return CORUN_EINVAL;
  const corun_moe_shape &s = *shape;
  if (s.hidden < 64 || s.hidden % 64 || s.n_experts < 1 || s.n_experts > MOE_MAX_EXPERTS || s.top_k < 1 ||
      s.top_k > MOE_MAX_TOPK || s.top_k > s.n_experts || s.expert_ffn < 64 || s.expert_ffn % 64 || s.n_shared < 0)
    return CORUN_EINVAL;
  corun_moe *m = new (std::nothrow) corun_moe();
  if (!m) return CORUN_ENOMEM;
  auto fail = [&](int rc) { corun_moe_destroy(m); return rc; };
  m->sh = s;
  m->B = B;
  m->BN = (B + 15) / 16 * 16;
  m->st = (cudaStream_t)cuda_stream;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&m->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return fail(CORUN_ECUDA);
  const int H = s.hidden, E = s.n_experts, F = s.expert_ffn, NB = E + s.n_shared;
  const size_t N1 = (size_t)NB * 2 * F, K2 = (size_t)NB * F;
  if (N1 > (size_t)1 << 30 || K2 > (size_t)1 << 30) return fail(CORUN_EINVAL);
  int rc;
  if ((rc = moe_alloc(m, &m->x_hi, (size_t)m->BN * H)) ||
      (rc = moe_alloc(m, &m->x_lo, (size_t)m->BN * H)) || (rc = moe_alloc(m, &m->h_hi, (size_t)m->BN * K2)) ||
      (rc = moe_alloc(m, &m->h_lo, (size_t)m->BN * K2)) ||
      (rc = moe_alloc(m, &m->out_gu, (size_t)m->BN * N1)) || (rc = moe_alloc(m, &m->out_d, (size_t)m->BN * H)) ||
      (rc = moe_alloc(m, &m->ws, gemm_ws_floats(m->num_sms, m->BN))) || (rc = moe_alloc(m, &m->w, (size_t)B * NB)) ||
      (rc = moe_alloc(m, &m->d_status, 1)))
    return fail(rc);
  m->router = (const bf16 *)router;
  // the three GEMMs run one after the other and their results are consumed in between: one workspace serves all
  // the form without groups: from 65 to 128 rows (used there only where the grouped form below does not apply) the
  // first GEMM applies the routing weight and the SwiGLU in its epilogue (where a tile width divides the experts'
  // width); else it stores gate / up sums and a kernel of its own follows (faster up to 64 rows, where the masked
  // store skips most of the output)
  const bool fused = m->BN > 64 && m->BN <= 128 && gemm_swiglu_blocks_half(F, NB, m->num_sms) > 0;
  if ((rc = fused ? gemm_plan_create_swiglu_blocks(&m->p_gu, gate_up, NB, F, H, m->x_hi, m->x_lo, B, m->BN, m->h_hi, m->h_lo, m->w, m->num_sms)
                  : gemm_plan_create(&m->p_gu, gate_up, (int)N1, H, m->x_hi, m->x_lo, B, m->BN, m->out_gu, m->ws, m->num_sms)) ||
      (rc = gemm_plan_create(&m->p_d, down, H, (int)K2, m->h_hi, m->h_lo, B, m->BN, m->out_d, m->ws, m->num_sms)))
    return fail(rc);
  if (!fused && (2 * F) % GEMM_TILE_N == 0) {       // a weight tile then belongs to one expert: skip the rows that
    m->p_gu.row_keep = m->w;                        // did not select it (the SwiGLU kernel does not read them)
    m->p_gu.keep_pitch = NB;
    m->p_gu.keep_div = 2 * F / GEMM_TILE_N;
  }
  // above 64 padded rows: the grouped form (one MMA per k-slice covers the hi and lo halves of a block of 64 rows,
  // where every row through every expert costs two on 128 rows), with the routing weight and the SwiGLU in the
  // per-group gate / up GEMM's epilogue
  const int g_half = gemm_swiglu_blocks_half(F, NB, m->num_sms);
  if (m->BN > 64 && g_half > 0 && H % GEMM_TILE_N == 0 && !getenv("CORUN_MOE_DECODE_DENSE")) {
    MoeGroups &g = m->grp;
    g.n_groups_max = moe_max_groups(B, E, s.n_shared, s.top_k);
    const size_t slots = (size_t)g.n_groups_max * MOE_GROUP_ROWS;
    if ((rc = moe_alloc(m, &g.tab_up, (size_t)g.n_groups_max * 3 + 1)) || (rc = moe_alloc(m, &g.tab_down, (size_t)g.n_groups_max * 3 + 1)) ||
        (rc = moe_alloc(m, &g.group_expert, (size_t)g.n_groups_max)) || (rc = moe_alloc(m, &g.slot_row, slots)) ||
        (rc = moe_alloc(m, &g.slot_of, (size_t)B * NB)) || (rc = moe_alloc(m, &g.slot_w, slots)) ||
        (rc = moe_alloc(m, &m->xg_hi, slots * H)) || (rc = moe_alloc(m, &m->xg_lo, slots * H)) ||
        (rc = moe_alloc(m, &m->hg_hi, slots * F)) || (rc = moe_alloc(m, &m->hg_lo, slots * F)) ||
        (rc = moe_alloc(m, &m->yg, slots * H)) || (rc = moe_alloc(m, &m->d_active, (size_t)B)))
      return fail(rc);
    std::vector<int> ones((size_t)B, 1);
    if (cudaMemcpy(m->d_active, ones.data(), (size_t)B * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return fail(CORUN_ECUDA);
    if ((rc = gemm_plan_create_grouped_swiglu(&m->p_gug, gate_up, (long long)NB * 2 * F, F, H, g_half, m->xg_hi, m->xg_lo, g.n_groups_max,
                                              MOE_GROUP_ROWS, m->hg_hi, m->hg_lo, g.slot_w, g.tab_up, m->num_sms)) ||
        (rc = gemm_plan_create_grouped(&m->p_dng, down, H, NB * F, H, F, m->hg_hi, m->hg_lo, g.n_groups_max, MOE_GROUP_ROWS, m->yg,
                                       g.tab_down, m->num_sms)))
      return fail(rc);
    m->grouped = true;
  }
  m->weight_bytes = ((int64_t)E * H + (int64_t)N1 * H + (int64_t)H * K2) * 2;
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(CORUN_ECUDA);
  *out = m;
  return CORUN_OK;
}

void corun_moe_destroy(corun_moe *m) {
  if (!m) return;
  cudaStreamSynchronize(m->st);
  gemm_plan_destroy(&m->p_gu);
  gemm_plan_destroy(&m->p_d);
  gemm_plan_destroy(&m->p_gug);
  gemm_plan_destroy(&m->p_dng);
  for (void *p : m->allocs) cudaFree(p);
  delete m;
}

int corun_moe_forward(corun_moe *m, const float *x, float *y, int32_t *experts, float *probs) {
  if (!m || !x || !y || x == y) return CORUN_EINVAL;
  if (((uintptr_t)y & 15u) || ((uintptr_t)x & 3u)) return CORUN_EINVAL;   // y is stored 16 bytes at a time
  const corun_moe_shape &s = m->sh;
  const int H = s.hidden, E = s.n_experts, F = s.expert_ffn, NB = E + s.n_shared;
  MCK(launch_split(x, m->B, H, m->x_hi, m->x_lo, m->st));
  MCK(launch_moe_router(m->x_hi, m->x_lo, H, m->router, m->B, E, s.n_shared, s.top_k, s.renormalize, m->w, experts, probs, m->st));
  if (m->grouped) {
    // rows grouped by expert -> gate / up with routing weight and SwiGLU, and down, per group -> the row's experts
    // summed in ascending expert id
    MCK(launch_moe_group(m->w, m->d_active, m->B, E, s.n_shared, F, m->grp, m->st));
    MCK(launch_moe_gather(m->x_hi, m->x_lo, H, m->grp, m->xg_hi, m->xg_lo, m->st));
    MCK(gemm_launch(m->p_gug, nullptr, m->d_status, m->st, nullptr, true));
    MCK(gemm_launch(m->p_dng, nullptr, m->d_status, m->st, nullptr, true));
    MCK(launch_moe_combine(m->yg, m->d_active, m->B, NB, H, m->grp, y, m->st));
    return CORUN_OK;
  }
  MCK(gemm_launch(m->p_gu, nullptr, m->d_status, m->st, nullptr, true));
  if (!m->p_gu.sw_hi) MCK(launch_moe_swiglu(m->p_gu.out(), m->w, m->B, F, NB, m->h_hi, m->h_lo, m->st));
  MCK(gemm_launch(m->p_d, nullptr, m->d_status, m->st, nullptr, true));
  MCK(launch_k(moe_readout_kernel, dim3((H / 4 + 255) / 256, m->B), dim3(256), 0, m->st, true, m->p_d.out(), H, y));
  return CORUN_OK;
}

int corun_moe_sync(corun_moe *m) {
  if (!m) return CORUN_EINVAL;
  int hs = 0;
  MCK(cudaMemcpyAsync(&hs, m->d_status, sizeof(int), cudaMemcpyDeviceToHost, m->st));
  MCK(cudaStreamSynchronize(m->st));
  return hs ? CORUN_ETIMEOUT : CORUN_OK;
}

int64_t corun_moe_weight_bytes(const corun_moe *m) { return m ? m->weight_bytes : 0; }

int corun_moe_launches(const corun_moe *m) { return m ? (m->grouped ? 7 : m->p_gu.sw_hi ? 5 : 6) : CORUN_EINVAL; }

}  // extern "C"
