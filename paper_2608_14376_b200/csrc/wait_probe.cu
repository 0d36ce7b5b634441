// Makes a bounded device-side wait run out, on purpose and harmlessly: one CTA waits, with the kernels' own
// wait routine and a limit the caller gives (a millisecond or so), on an mbarrier that nothing ever arrives at.
// The wait gives up, the kernel records the code in a status word and returns normally; the host reports
// CORUN_ETIMEOUT.  No trap, no fault, no unbounded spin: the context stays usable, which the test checks by
// running an ordinary kernel afterwards.  Also hosts corun_debug_check_index (the index checks of checks.cuh
// evaluated on the host, for the unit tests).
#include <cuda_runtime.h>

#include "../../include/corun.h"
#include "../../include/corun_debug.h"
#include "checks.cuh"
#include "gemm.cuh"
#include "ptx.cuh"

using namespace corun;

namespace {

__global__ void __launch_bounds__(32) wait_probe_kernel(unsigned long long limit_ns, int *status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    // phase 0 never completes: no thread arrives, no copy is in flight
    const bool ok = mbar_wait_limit(smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (!ok) atomicCAS(status, 0, DEV_TIMEOUT_EPILOGUE);
  }
}

}  // namespace

extern "C" int corun_debug_wait_probe(uint64_t limit_ns, void *cuda_stream) {
  if (limit_ns < 1000 || limit_ns > 100000000ull) return CORUN_EINVAL;   // 1 us .. 100 ms: never a long stall
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int *d = nullptr;
  if (cudaMalloc(&d, sizeof(int)) != cudaSuccess) return CORUN_ENOMEM;
  int hs = 0;
  cudaError_t ce = cudaMemsetAsync(d, 0, sizeof(int), st);
  if (ce == cudaSuccess) {
    wait_probe_kernel<<<1, 32, 0, st>>>(limit_ns, d);
    ce = cudaGetLastError();
  }
  if (ce == cudaSuccess) ce = cudaMemcpyAsync(&hs, d, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
  cudaFree(d);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return hs != 0 ? CORUN_ETIMEOUT : CORUN_OK;
}

extern "C" int corun_debug_check_index(int32_t kind, int64_t a, int64_t b, int64_t c, int64_t d, int64_t e, int64_t f, int64_t g) {
  switch (kind) {
    case 0: return check_slot_pos(a, b, c, d, e) ? 1 : 0;
    case 1: return check_page(a, b) ? 1 : 0;
    case 2: return check_item(a, b, c, d, e, f, g) ? 1 : 0;
    case 3: return check_ws_slot(a, b, c) ? 1 : 0;
    default: return CORUN_EINVAL;
  }
}
