// Launchers of the Mixture-of-Experts kernels (moe.cu) for the engine's row program.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "gemm.cuh"

namespace corun {

// Softmax over the E router logits of every row (columns 0..E-1 of `logits`), top_k by repeated arg-max with
// ties to the lower id, optional renormalisation; writes the row of SwiGLU weights w[r, 0 .. E + S) (p_e for
// the selected experts, 0 for the others, 1 for the shared ones) and, when not null, the routing.
cudaError_t launch_moe_route(const GemmOut &logits, int R, int E, int S, int top_k, int renormalize, float *w,
                             int *experts, float *probs, cudaStream_t st);
// h[r, e*F + f] = w[r, e] * silu(gate) * up as a bf16 hi/lo pair (zeros where w[r, e] == 0); gate / up are
// columns e*2F + f and e*2F + F + f of `gu`; n_blocks = E + S.
cudaError_t launch_moe_swiglu(const GemmOut &gu, const float *w, int R, int F, int n_blocks, __nv_bfloat16 *out_hi,
                              __nv_bfloat16 *out_lo, cudaStream_t st);

}  // namespace corun
