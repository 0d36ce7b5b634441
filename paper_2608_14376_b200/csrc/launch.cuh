// Kernel launch helper: every kernel of the row program is launched with programmatic stream
// serialization, so that its prologue (and, for the GEMM, the first weight tiles, which depend on
// nothing) overlaps the tail of its predecessor.  Each such kernel executes griddepcontrol.wait
// before it touches anything a predecessor produces or still reads.
#pragma once
#include <cuda_runtime.h>

namespace corun {

extern bool g_use_pdl;   // false when the environment sets CORUN_NO_PDL=1

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                            Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pdl && g_use_pdl) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace corun
