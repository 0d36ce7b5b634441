// Launchers of the Mixture-of-Experts kernels (moe.cu) for the engine's row program.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "gemm.cuh"

namespace corun {

// Router of every row: logits = Wr x (Wr bf16 [E, H]; x the row's bf16 hi + lo pair, [R or more, H]) on the CUDA
// cores, softmax over all E experts, top_k by repeated arg-max with ties to the lower id, optional
// renormalisation; writes the row of SwiGLU weights w[r, 0 .. E + S) (p_e for the selected experts, 0 for the
// others, 1 for the shared ones) and, when not null, the routing.  One CTA per row; H * 4 bytes of shared memory
// (H <= 12288).
cudaError_t launch_moe_router(const __nv_bfloat16 *x_hi, const __nv_bfloat16 *x_lo, int H, const __nv_bfloat16 *Wr, int R, int E,
                              int S, int top_k, int renormalize, float *w, int *experts, float *probs, cudaStream_t st);
// h[r, e*F + f] = w[r, e] * silu(gate) * up as a bf16 hi/lo pair (zeros where w[r, e] == 0); gate / up are
// columns e*2F + f and e*2F + F + f of `gu`; n_blocks = E + S.
cudaError_t launch_moe_swiglu(const GemmOut &gu, const float *w, int R, int F, int n_blocks, __nv_bfloat16 *out_hi,
                              __nv_bfloat16 *out_lo, cudaStream_t st);

// ---- grouped form (prefill chunks): every expert's rows gathered into blocks of MOE_GROUP_ROWS rows ----
constexpr int MOE_GROUP_ROWS = 64;
// Most groups a chunk of R rows can need: one per expert plus one per full block of selected (row, expert) pairs.
inline int moe_max_groups(int R, int E, int S, int top_k) { return E + S + R * (top_k + S) / MOE_GROUP_ROWS; }

// Buffers of the grouped form (device, owned by the caller).
struct MoeGroups {
  int n_groups_max;      // moe_max_groups(...)
  int *tab_up;           // [n_groups_max][3] + 1: first gate/up weight row (e * 2F), 0, rows   (gemm group table);
                         //   the last int: groups in use
  int *tab_down;         // [n_groups_max][3] + 1: 0, first down k-block (e * F / 64), rows; groups in use
  int *group_expert;     // [n_groups_max]
  int *slot_row;         // [n_groups_max * 64]: the chunk row gathered into the slot (valid below the group's row count)
  int *slot_of;          // [E + S][R]: where the row sits in the expert's groups, -1 = not selected
  float *slot_w;         // [n_groups_max * 64]: the slot's routing weight w[row, expert] (valid below the group's row count)
};

// Groups the chunk's (row, expert) pairs: experts ascending, an expert's rows ascending, 64 per group; rows with
// active[r] == 0 are left out.  w: the routing weights [R][E + S] of launch_moe_route.  One CTA.
cudaError_t launch_moe_group(const float *w, const int *active, int R, int E, int S, int F, const MoeGroups &g,
                             cudaStream_t st);
// xg[slot, :] = x[slot_row[slot], :] for both halves of the activations (bf16, H values per row).
cudaError_t launch_moe_gather(const __nv_bfloat16 *x_hi, const __nv_bfloat16 *x_lo, int H, const MoeGroups &g,
                              __nv_bfloat16 *xg_hi, __nv_bfloat16 *xg_lo, cudaStream_t st);
// hg[slot, f] = w[row, expert] * silu(gate) * up from the grouped gate/up result gu [slots][2F] (plain matrix).
cudaError_t launch_moe_swiglu_grouped(const float *gu, const float *w, int n_blocks, int F, const MoeGroups &g,
                                      __nv_bfloat16 *hg_hi, __nv_bfloat16 *hg_lo, cudaStream_t st);
// y[r, :] = sum over the row's experts in ascending expert id (shared experts last) of yg[slot_of[r, e], :];
// rows that are not active are left alone.
cudaError_t launch_moe_combine(const float *yg, const int *active, int R, int n_blocks, int H, const MoeGroups &g, float *y,
                               cudaStream_t st);

}  // namespace corun
