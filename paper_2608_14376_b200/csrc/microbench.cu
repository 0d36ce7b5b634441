// Micro-benchmark of three reductions with a tiling that is FIXED for every batch size against a tiling that
// ADAPTS to it (the paper's motivation, Introduction and Fig. 2: batch-invariant kernels pay for using one
// tiling everywhere; a position-invariant path only has to keep the tiling fixed for its one padded shape).
//   kind 0  RMSNorm of every row of x [R, N]            y [R, N]
//   kind 1  softmax of every row of x [R, N]            y [R, N]
//   kind 2  sum over the R rows of x [R, N]             y [N]      (a reduction ACROSS the batch)
//   variant 0  fixed: one CTA of 256 threads per row (kinds 0, 1) or per 256 columns with the rows added in
//              ascending order (kind 2), whatever R is: a result's bits do not depend on R;
//   variant 1  adaptive: with few rows, a row is split over a cluster of up to 8 CTAs whose partial results
//              meet in distributed shared memory (kinds 0, 1: the summation tree changes with R); the rows are
//              split over as many CTAs as fill the GPU and their partial sums are added with atomics (kind 2:
//              the order is not even fixed from run to run).
// Not part of the decode path: measurement only.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "../../include/corun.h"
#include "../../include/corun_debug.h"
#include "gemm.cuh"

namespace cg = cooperative_groups;
using namespace corun;

namespace {

constexpr int MB_THREADS = 256;

// Block-wide sum / max in one fixed order: thread-serial, xor butterfly, warp results ascending.
__device__ __forceinline__ float mb_block_sum(float v, float *scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < MB_THREADS / 32; ++w) t += scratch[w];
  return t;
}
__device__ __forceinline__ float mb_block_max(float v, float *scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = -CUDART_INF_F;
  for (int w = 0; w < MB_THREADS / 32; ++w) t = fmaxf(t, scratch[w]);
  return t;
}

// A value of every CTA of the cluster combined in rank order (C = 1: the value itself).
template <bool IS_MAX>
__device__ __forceinline__ float mb_cluster_combine(float v, float *slot, int C) {
  if (C == 1) return v;
  cg::cluster_group cl = cg::this_cluster();
  if (threadIdx.x == 0) *slot = v;
  cl.sync();
  float t = IS_MAX ? -CUDART_INF_F : 0.f;
  for (int c = 0; c < C; ++c) {
    const float o = *cl.map_shared_rank(slot, c);
    t = IS_MAX ? fmaxf(t, o) : t + o;
  }
  cl.sync();                                          // nobody overwrites its slot before all have read it
  return t;
}

// Row r = blockIdx.x / C; CTA c of its cluster takes columns [c * N / C, (c + 1) * N / C)  (N % (4 * C) == 0).
__global__ void __launch_bounds__(MB_THREADS) mb_rmsnorm_kernel(const float *__restrict__ x, int N, int C, float eps, float *__restrict__ y) {
  __shared__ float scratch[MB_THREADS / 32];
  __shared__ float slot;
  const int r = blockIdx.x / C, c = blockIdx.x % C, n0 = c * (N / C), n1 = n0 + N / C;
  const float *xr = x + (size_t)r * N;
  float ss = 0.f;
  for (int i = n0 + 4 * threadIdx.x; i < n1; i += 4 * MB_THREADS) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + i);
    ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
  }
  const float tot = mb_cluster_combine<false>(mb_block_sum(ss, scratch), &slot, C);
  const float inv = rsqrtf(tot / (float)N + eps);
  for (int i = n0 + 4 * threadIdx.x; i < n1; i += 4 * MB_THREADS) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + i);
    *reinterpret_cast<float4 *>(y + (size_t)r * N + i) = make_float4(v.x * inv, v.y * inv, v.z * inv, v.w * inv);
  }
}

__global__ void __launch_bounds__(MB_THREADS) mb_softmax_kernel(const float *__restrict__ x, int N, int C, float *__restrict__ y) {
  __shared__ float scratch[MB_THREADS / 32];
  __shared__ float slot;
  const int r = blockIdx.x / C, c = blockIdx.x % C, n0 = c * (N / C), n1 = n0 + N / C;
  const float *xr = x + (size_t)r * N;
  float mx = -CUDART_INF_F;
  for (int i = n0 + 4 * threadIdx.x; i < n1; i += 4 * MB_THREADS) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + i);
    mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
  }
  mx = mb_cluster_combine<true>(mb_block_max(mx, scratch), &slot, C);
  float sum = 0.f;
  for (int i = n0 + 4 * threadIdx.x; i < n1; i += 4 * MB_THREADS) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + i);
    sum += __expf(v.x - mx); sum += __expf(v.y - mx); sum += __expf(v.z - mx); sum += __expf(v.w - mx);
  }
  const float inv = 1.f / mb_cluster_combine<false>(mb_block_sum(sum, scratch), &slot, C);
  for (int i = n0 + 4 * threadIdx.x; i < n1; i += 4 * MB_THREADS) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + i);
    *reinterpret_cast<float4 *>(y + (size_t)r * N + i) =
        make_float4(__expf(v.x - mx) * inv, __expf(v.y - mx) * inv, __expf(v.z - mx) * inv, __expf(v.w - mx) * inv);
  }
}

// Column sums.  blockIdx.x: block of 256 columns; blockIdx.y: chunk of rows [y * rows_per, ...).  One chunk (fixed):
// plain stores, rows ascending.  Several chunks (adaptive): partial sums added with atomics into a zeroed y.
__global__ void __launch_bounds__(MB_THREADS) mb_colsum_kernel(const float *__restrict__ x, int R, int N, int rows_per, float *__restrict__ y) {
  const int n = blockIdx.x * MB_THREADS + threadIdx.x;
  if (n >= N) return;
  const int r0 = blockIdx.y * rows_per, r1 = min(R, r0 + rows_per);
  float acc = 0.f;
  for (int r = r0; r < r1; ++r) acc += x[(size_t)r * N + n];
  if (gridDim.y == 1) y[n] = acc;
  else atomicAdd(y + n, acc);
}

cudaError_t mb_launch_rows(int kind, const float *x, int R, int N, int C, float *y, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(R * C);
  cfg.blockDim = dim3(MB_THREADS);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (kind == 0) return cudaLaunchKernelEx(&cfg, mb_rmsnorm_kernel, x, N, C, 1e-6f, y);
  return cudaLaunchKernelEx(&cfg, mb_softmax_kernel, x, N, C, y);
}

}  // namespace

extern "C" int corun_debug_microbench(int32_t kind, int32_t variant, const float *x, int32_t R, int32_t N, float *y,
                                      int32_t reps, float *avg_us, int32_t *tiling, void *cuda_stream) {
  if (!x || !y || kind < 0 || kind > 2 || variant < 0 || variant > 1 || R < 1 || N < 32 || N % 32 || reps < 1) return CORUN_EINVAL;
  if (((uintptr_t)x & 15u) || ((uintptr_t)y & 15u)) return CORUN_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int dev = 0, sms = 0;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (ce != cudaSuccess || sms < 1) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  // the adaptive choice: enough CTAs to fill the GPU about twice
  int C = 1, chunks = 1;
  if (variant == 1 && kind < 2) {
    while (C < 8 && R * C * 2 <= 2 * sms && N % (8 * C) == 0) C *= 2;
  } else if (variant == 1) {
    const int col_blocks = (N + MB_THREADS - 1) / MB_THREADS;
    chunks = 2 * sms / col_blocks;
    if (chunks > R / 4) chunks = R / 4;
    if (chunks < 1) chunks = 1;
  }
  if (tiling) *tiling = kind < 2 ? C : chunks;
  const int rows_per = (R + chunks - 1) / chunks;
  auto once = [&]() -> cudaError_t {
    if (kind < 2) return mb_launch_rows(kind, x, R, N, C, y, st);
    if (chunks > 1) {
      cudaError_t e = cudaMemsetAsync(y, 0, (size_t)N * sizeof(float), st);
      if (e != cudaSuccess) return e;
    }
    mb_colsum_kernel<<<dim3((N + MB_THREADS - 1) / MB_THREADS, (R + rows_per - 1) / rows_per), MB_THREADS, 0, st>>>(x, R, N, rows_per, y);
    return cudaGetLastError();
  };
  cudaEvent_t e0, e1;
  ce = cudaEventCreate(&e0);
  if (ce == cudaSuccess) ce = cudaEventCreate(&e1);
  if (ce == cudaSuccess) ce = once();                 // warm-up
  if (ce == cudaSuccess) ce = cudaEventRecord(e0, st);
  for (int i = 0; i < reps && ce == cudaSuccess; ++i) ce = once();
  if (ce == cudaSuccess) ce = cudaEventRecord(e1, st);
  if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
  float ms = 0.f;
  if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  if (avg_us) *avg_us = ms * 1e3f / (float)reps;
  return CORUN_OK;
}
