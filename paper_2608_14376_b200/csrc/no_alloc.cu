// corun_gemm_static: the stand-alone GEMM for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they
// need a GEMM: code that runs inside a memory-pool or arena that owns all
// device memory up front, a real-time loop where an allocation's implicit
// device synchronisation is not acceptable, or a process whose memory budget
// was handed out at start-up.  For them the split activations, the per-CTA
// partial sums, the partition tables and the status word live in one
// file-scope device array of fixed size, reserved by every GPU that loads the
// library until the process exits.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "../../include/corun.h"
#include "gemm.cuh"
#include "ops.cuh"

using namespace corun;

namespace {

constexpr int NA_MAX_R = CORUN_STATIC_MAX_ROWS;
constexpr int NA_MAX_K = CORUN_STATIC_MAX_K;
constexpr int NA_MAX_N = CORUN_STATIC_MAX_N;
constexpr int NA_MAX_GRID = 192;                 // CTAs (= SMs) the partial-sum area is sized for
constexpr int NA_BN = 16;                        // padded row count of the MMA's N operand
constexpr int NA_MAX_TILES = NA_MAX_N / GEMM_TILE_N;

constexpr size_t NA_OFF_HI = 0;
constexpr size_t NA_HILO_BYTES = (size_t)NA_BN * NA_MAX_K * sizeof(__nv_bfloat16);
constexpr size_t NA_OFF_LO = NA_OFF_HI + NA_HILO_BYTES;
constexpr size_t NA_OFF_WS = NA_OFF_LO + NA_HILO_BYTES;
constexpr size_t NA_WS_BYTES = (size_t)NA_MAX_GRID * 2 * NA_BN * GEMM_TILE_N * sizeof(float);
constexpr size_t NA_OFF_TAB = NA_OFF_WS + NA_WS_BYTES;
constexpr int NA_TAB_INTS = NA_MAX_GRID + 1 + 3 * NA_MAX_TILES;
constexpr size_t NA_TAB_BYTES = ((size_t)NA_TAB_INTS * sizeof(int) + 255) / 256 * 256;
constexpr size_t NA_OFF_STATUS = NA_OFF_TAB + NA_TAB_BYTES;
constexpr size_t NA_BYTES = NA_OFF_STATUS + 256;

// The scratch itself (about 6.3 MiB per GPU).  In host code this name is only
// a handle for cudaGetSymbolAddress; kernels get the address obtained there.
static __device__ __align__(256) unsigned char g_static_scratch[NA_BYTES];

constexpr int NA_MAX_DEVICES = 64;
// Per-device cache of the set-up.  The address is published last (release) and read first (acquire), so a
// thread that sees it also sees the SM count written before it; two threads that both find it empty do the
// same idempotent set-up and store the same values.
std::atomic<unsigned char *> g_scratch_addr[NA_MAX_DEVICES];
int g_num_sms[NA_MAX_DEVICES] = {0};

// One-time set-up per device (the device must be current): resolves the
// device address of the scratch array and opts the GEMM kernel into its
// shared-memory size.  Allocates nothing.
int static_setup(int dev, unsigned char **base, int *sms) {
  if (dev < 0 || dev >= NA_MAX_DEVICES) return CORUN_EINVAL;
  unsigned char *cached = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!cached) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) { g_last_cuda_error = (int)e; return CORUN_ECUDA; }
    int n = 0;
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = gemm_prepare_kernel();
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return CORUN_ECUDA; }
    if (n < 1) return CORUN_ECUDA;
    g_num_sms[dev] = n;
    cached = (unsigned char *)p;
    g_scratch_addr[dev].store(cached, std::memory_order_release);
  }
  *base = cached;
  *sms = g_num_sms[dev];
  return *sms >= 1 ? CORUN_OK : CORUN_ECUDA;
}

}  // namespace

extern "C" int corun_gemm_static(const void *W, int32_t N, int32_t K, const float *X, int32_t R, float *out,
                                 void *cuda_stream) {
  if (!W || !X || !out || N < 1 || K < 64 || K % 64 || R < 1) return CORUN_EINVAL;
  // the kernels store the output 16 bytes at a time and read W through a tensor map: a buffer that starts
  // elsewhere (a view into an arena, say) would fault on the device, so it is refused here, before any launch
  if (((uintptr_t)out & 15u) || ((uintptr_t)W & 15u) || ((uintptr_t)X & 3u)) return CORUN_EINVAL;
  if (R > NA_MAX_R || K > NA_MAX_K || N > NA_MAX_N) return CORUN_ELIMIT;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  {
    // every call ends with a stream synchronisation and a copy of the status word to the host, neither of which
    // a capturing stream permits: refuse instead of breaking the caller's capture
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs != cudaStreamCaptureStatusNone) return CORUN_EINVAL;
  }
  int dev = 0;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  unsigned char *base = nullptr;
  int sms = 0;
  int rc = static_setup(dev, &base, &sms);
  if (rc != CORUN_OK) return rc;
  if (sms > NA_MAX_GRID) return CORUN_ELIMIT;

  __nv_bfloat16 *hi = (__nv_bfloat16 *)(base + NA_OFF_HI), *lo = (__nv_bfloat16 *)(base + NA_OFF_LO);
  float *ws = (float *)(base + NA_OFF_WS);
  int *tab = (int *)(base + NA_OFF_TAB);
  int *status = (int *)(base + NA_OFF_STATUS);

  // the same static partition as the allocating path, with its tables built on the stack
  GemmPlan p;
  int host_tab[NA_TAB_INTS];
  int n_ints = 0;
  if ((rc = gemm_plan_fill(&p, W, N, K, hi, lo, R, NA_BN, out, ws, sms, host_tab, NA_TAB_INTS, &n_ints)) != 0) return rc;
  gemm_plan_bind_tables(&p, tab);

  // The array keeps whatever the previous call left: clear what must start at
  // zero (padding rows of the split activations, the status word).
  ce = cudaMemsetAsync(base + NA_OFF_HI, 0, 2 * NA_HILO_BYTES, st);
  if (ce == cudaSuccess) ce = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (ce == cudaSuccess) ce = cudaMemcpyAsync(tab, host_tab, (size_t)n_ints * sizeof(int), cudaMemcpyHostToDevice, st);
  if (ce == cudaSuccess) ce = launch_split(X, R, K, hi, lo, st);
  if (ce == cudaSuccess) ce = gemm_launch(p, nullptr, status, st);
  if (ce == cudaSuccess) ce = gemm_fixup_launch(p, st);
  int hs = 0;
  if (ce == cudaSuccess) ce = cudaMemcpyAsync(&hs, status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return hs != 0 ? CORUN_ETIMEOUT : CORUN_OK;
}
