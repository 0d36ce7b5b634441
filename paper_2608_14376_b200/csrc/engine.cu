// Host side of the C ABI: engine state, paged KV pool, the row program
// (decode graph / eager prefill) and the debug accessors.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/corun.h"
#include "../../include/corun_debug.h"
#include "gemm.cuh"
#include "mla.cuh"
#include "moe.cuh"
#include "ops.cuh"

using namespace corun;


#define CK(call)                                   \
  do {                                             \
    cudaError_t _e = (call);                       \
    if (_e != cudaSuccess) {                       \
      g_last_cuda_error = (int)_e;                 \
      return CORUN_ECUDA;                          \
    }                                              \
  } while (0)
#define RC(call)                  \
  do {                            \
    int _r = (call);              \
    if (_r != CORUN_OK) return _r; \
  } while (0)

namespace {

typedef __nv_bfloat16 bf16;

// Buffers and GEMM plans of the row program at one fixed row count.
struct Program {
  int R = 0, BN = 0;
  float *h = nullptr, *q = nullptr, *part_acc = nullptr, *part_ml = nullptr;
  float *qkv_out = nullptr, *o_out = nullptr, *gu_out = nullptr, *down_out = nullptr, *logits = nullptr, *ws = nullptr;
  bf16 *xn_hi = nullptr, *xn_lo = nullptr, *ao_hi = nullptr, *ao_lo = nullptr, *ff_hi = nullptr, *ff_lo = nullptr;
  int *row_token = nullptr, *row_pos = nullptr, *row_active = nullptr, *row_slot = nullptr, *do_sample = nullptr;
  int *row_blocks = nullptr;   // decode program: which blocks of rows hold a request this step (GemmPlan::row_blocks)
  // decode program: the step's rows are the slots with a request first (prepare_rows); the slot's row, and the
  // slots' sampling state at the rows' places
  int *slot_row = nullptr, *row_step = nullptr;
  float *row_temp = nullptr, *row_top_p = nullptr;
  int *sampled = nullptr, *att_work = nullptr, *att_n_work = nullptr, *att_pool = nullptr;
  GemmPlan p_qkv, p_o, p_gu, p_down, p_lm;
  // Mixture-of-Experts feed-forward layers: p_gu / p_down are then the GEMMs over all experts' gate / up rows
  // and over the concatenated hidden activations; moe_w the rows' routing weights
  float *moe_w = nullptr;
  // grouped form of the experts' GEMMs (prefill chunks: the rows of an expert gathered into blocks of 64)
  bool grouped = false;
  MoeGroups grp{};
  GemmPlan p_gug, p_dng;
  bf16 *xg_hi = nullptr, *xg_lo = nullptr, *hg_hi = nullptr, *hg_lo = nullptr;
  float *gug_out = nullptr, *yg_out = nullptr;
  int *plain_tiles = nullptr;            // zeros: the table that makes a plain matrix readable as a GEMM result
  // multi-head latent attention: head-major matrices of RPH rows per head for the grouped up-projections
  // (p_uk: q_lat = W_uk^T q_nope; p_uv: [. | o] = W_kv_b o_lat), the attention's partials, and the dense
  // feed-forward GEMMs of the layers that have no experts
  int RPH = 0;
  bf16 *qn_hi = nullptr, *qn_lo = nullptr, *ol_hi = nullptr, *ol_lo = nullptr;
  float *q_lat = nullptr, *q_rope = nullptr, *uv_out = nullptr, *mla_po = nullptr;
  float2 *mla_ml = nullptr;
  int *tab_uk = nullptr, *tab_uv = nullptr;
  GemmPlan p_uk, p_uv, p_gu_d, p_down_d;
  bool has_layers = false, has_lm = false;
  std::vector<void *> allocs;
};

}  // namespace

struct corun_engine {
  corun_shape sh{};
  int B = 0, max_ctx = 0, max_blocks = 0, max_splits = 0, chunk = 0, num_sms = 0;
  int whole_pairs = 0;               // ablation: attention without parallelism inside a (row, kv head) pair
  int64_t pool_blocks = 0;
  cudaStream_t st = nullptr;
  bool own_stream = false;
  const void *w0_qkv = nullptr, *w0_o = nullptr, *w0_gu = nullptr, *w0_down = nullptr;
  // borrowed weights
  const bf16 *embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  std::vector<const bf16 *> attn_norm, mlp_norm;
  std::vector<CUtensorMap> tm_qkv, tm_o, tm_gu, tm_down;
  std::vector<CUtensorMap> tm_gu_half;     // dense gate / up matrices with the box of the GEMM with SwiGLU in its epilogue
  std::vector<CUtensorMap> tm_k, tm_v;   // per layer: the pages as rows of head_dim halfs (keys and values alike)
  std::vector<CUtensorMap> tm_k4;        // the same memory as [8-token group][64-dim half][8 tokens][64 dims]: one box per (page, head) tile
  // Mixture-of-Experts feed-forward layers (E = 0: dense).  sh.ffn is then (E + S) * F.
  int moe_E = 0, moe_K = 0, moe_F = 0, moe_S = 0, moe_renorm = 0;
  std::vector<const bf16 *> router;      // per layer: [E, H], borrowed
  // multi-head latent attention (corun_init_mla): sh.head_dim is the value width, the cache holds rank + rope
  // halfs per token; layers below first_dense have a dense feed-forward of width dense_ffn
  bool mla = false;
  MlaDims md{};
  int first_dense = 0, dense_ffn = 0, mla_splits = 0;
  std::vector<const bf16 *> kv_norm;
  bf16 *w_ukT = nullptr;                 // [L][nh * rank][nope]: the key up-projections transposed
  std::vector<CUtensorMap> tm_uk, tm_uv, tm_c, tm_cv, tm_gu_d, tm_down_d;
  const void *w0_uv = nullptr, *w0_gu_d = nullptr, *w0_down_d = nullptr;
  // KV
  __half *kv_pool = nullptr;
  size_t layer_stride = 0;
  int *d_block_table = nullptr;
  // Pages are handed out in aligned runs of kv_run consecutive pool pages (1; 4 for latent caches created with
  // kv_block = 64: the latent attention kernel then fetches a run with one TMA box).  free_blocks / slot_blocks hold
  // RUN indices; the block table holds pages (run * kv_run + i).
  int kv_run = 1;
  std::vector<int> free_blocks;
  std::vector<std::vector<int>> slot_blocks;
  float2 *d_rope = nullptr;
  // slot state: device
  int *d_in_use = nullptr, *d_ctx = nullptr, *d_step = nullptr, *d_pending = nullptr;
  float *d_temp = nullptr, *d_top_p = nullptr;
  float *pf_logits = nullptr;            // [B, vocab]: a slot's logits after its prefill (the decode logits are by row)
  std::vector<int> logits_row;           // per slot: its row of the last decode step it took part in, -1 = pf_logits
  uint64_t *d_seeds = nullptr;
  uint8_t *d_active = nullptr;
  int *d_out_tokens = nullptr, *d_status = nullptr;
  // slot state: host mirrors
  std::vector<int> in_use, ctx, reserve, step;
  // pinned staging
  uint8_t *h_active = nullptr;
  uint64_t *h_seeds = nullptr;
  int *h_out_tokens = nullptr, *h_status = nullptr;
  int *h_rows = nullptr;          // prefill row metadata staging [5][chunk]
  bool staged_valid = false, in_flight = false;
  Program dec, pre, lm1;
  // prefill-only per-row sampling arrays (length 1)
  float *d_pf_temp = nullptr, *d_pf_top_p = nullptr;
  uint64_t *d_pf_seed = nullptr;
  int *d_pf_step = nullptr, *d_pf_one = nullptr, *d_pf_tok = nullptr;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t graph_exec = nullptr;
  bool eager = false;
  unsigned long long *step_trace = nullptr;   // debug (CORUN_TRACE_STEP=1): GEMM timelines of a whole step
  int stop_after = -1;            // debug: eager decode stops after this many stages of layer 0
  int decode_launches = 0;
  std::vector<void *> allocs;
};

namespace {

template <typename T>
int dmalloc(std::vector<void *> &keep, T **p, size_t n, bool zero = true) {
  void *q = nullptr;
  if (n == 0) n = 1;
  cudaError_t e = cudaMalloc(&q, n * sizeof(T));
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return CORUN_ENOMEM;
  }
  keep.push_back(q);
  if (zero && cudaMemset(q, 0, n * sizeof(T)) != cudaSuccess) return CORUN_ECUDA;
  *p = (T *)q;
  return CORUN_OK;
}

int pad16(int x) { return (x + 15) / 16 * 16; }

// fuse_swiglu: the gate / up GEMM writes silu(gate) * up itself (dense feed-forward, up to 128 padded rows: the
// decode program while it is bound by the weight stream; whole tiles on fewer CTAs would cost a prefill chunk,
// which is bound by the tensor pipe, a third of its gate / up rate).
int program_create(corun_engine *e, Program &P, int R, bool layers, bool lm, bool grouped = false, bool fuse_swiglu = false) {
  const corun_shape &s = e->sh;
  const int H = s.hidden, QD = s.n_q_heads * s.head_dim, KD = s.n_kv_heads * s.head_dim, F = s.ffn, V = s.vocab;
  const MlaDims &md = e->md;
  // columns of the q / k / v (MLA: q / kv_a) projection
  const int QKVN = e->mla ? md.nh * (md.nope + md.rope) + md.rank + md.rope : QD + 2 * KD;
  const int Fd = e->dense_ffn;                      // MLA: width of the dense feed-forward layers beside expert layers
  const int Fmax = F > Fd ? F : Fd;
  P.R = R;
  P.BN = pad16(R);
  P.has_layers = layers;
  P.has_lm = lm;
  auto &A = P.allocs;
  RC(dmalloc(A, &P.xn_hi, (size_t)P.BN * H));
  RC(dmalloc(A, &P.xn_lo, (size_t)P.BN * H));
  RC(dmalloc(A, &P.ws, gemm_ws_floats(e->num_sms, P.BN)));
  RC(dmalloc(A, &P.row_token, R));
  RC(dmalloc(A, &P.row_pos, R));
  RC(dmalloc(A, &P.row_active, R));
  RC(dmalloc(A, &P.row_slot, R));
  RC(dmalloc(A, &P.do_sample, R));
  RC(dmalloc(A, &P.sampled, R));
  RC(dmalloc(A, &P.row_blocks, 1));
  RC(dmalloc(A, &P.slot_row, R));
  RC(dmalloc(A, &P.row_step, R));
  RC(dmalloc(A, &P.row_temp, R));
  RC(dmalloc(A, &P.row_top_p, R));
  if (layers) {
    RC(dmalloc(A, &P.h, (size_t)R * H));
    if (!e->mla) {
      RC(dmalloc(A, &P.q, (size_t)R * QD));
      RC(dmalloc(A, &P.part_acc, (size_t)R * s.n_q_heads * e->max_splits * s.head_dim));
      RC(dmalloc(A, &P.part_ml, (size_t)R * s.n_q_heads * e->max_splits * 2));
      RC(dmalloc(A, &P.att_work, (size_t)R * e->max_splits * e->sh.n_kv_heads));
      RC(dmalloc(A, &P.att_n_work, 2 + 2 * (size_t)R * e->sh.n_kv_heads));
      RC(dmalloc(A, &P.att_pool, (size_t)s.n_layers));
    } else {
      const int BG = mla_group_rows(P.BN), n_groups = md.nh * (mla_rows_per_head(P.BN) / BG);
      P.RPH = mla_rows_per_head(P.BN);
      const size_t hr = (size_t)md.nh * P.RPH;      // rows of the head-major matrices
      RC(dmalloc(A, &P.qn_hi, hr * md.nope));
      RC(dmalloc(A, &P.qn_lo, hr * md.nope));
      RC(dmalloc(A, &P.q_lat, hr * md.rank));
      RC(dmalloc(A, &P.q_rope, (size_t)R * md.nh * md.rope));
      RC(dmalloc(A, &P.ol_hi, hr * md.rank));
      RC(dmalloc(A, &P.ol_lo, hr * md.rank));
      RC(dmalloc(A, &P.uv_out, hr * (md.nope + md.vh)));
      RC(dmalloc(A, &P.mla_ml, (size_t)mla_part_ml_floats(R, md.nh, e->max_ctx) / 2));
      RC(dmalloc(A, &P.mla_po, (size_t)mla_part_o_floats(R, md.nh, md.rank, e->max_ctx)));
      RC(dmalloc(A, &P.tab_uk, (size_t)n_groups * 3 + 1));
      RC(dmalloc(A, &P.tab_uv, (size_t)n_groups * 3 + 1));
      std::vector<int> tk((size_t)n_groups * 3 + 1), tv((size_t)n_groups * 3 + 1);
      tk[(size_t)n_groups * 3] = tv[(size_t)n_groups * 3] = n_groups;   // all groups are in use
      for (int g = 0; g < n_groups; ++g) {          // group = (head, block of BG rows): its weight rows, rows in use
        const int h = g / (P.RPH / BG), rb = g % (P.RPH / BG);
        const int valid = R - rb * BG < BG ? (R - rb * BG > 0 ? R - rb * BG : 0) : BG;
        tk[3 * g] = h * md.rank; tk[3 * g + 1] = 0; tk[3 * g + 2] = valid;
        tv[3 * g] = h * (md.nope + md.vh); tv[3 * g + 1] = 0; tv[3 * g + 2] = valid;
      }
      CK(cudaMemcpy(P.tab_uk, tk.data(), tk.size() * sizeof(int), cudaMemcpyHostToDevice));
      CK(cudaMemcpy(P.tab_uv, tv.data(), tv.size() * sizeof(int), cudaMemcpyHostToDevice));
      RC(gemm_plan_create_grouped(&P.p_uk, e->w_ukT, (long long)md.nh * md.rank, md.nope, md.rank, md.nope, P.qn_hi, P.qn_lo, n_groups,
                                  BG, P.q_lat, P.tab_uk, e->num_sms));
      RC(gemm_plan_create_grouped(&P.p_uv, e->w0_uv, (long long)md.nh * (md.nope + md.vh), md.rank, md.nope + md.vh, md.rank, P.ol_hi,
                                  P.ol_lo, n_groups, BG, P.uv_out, P.tab_uv, e->num_sms));
      P.p_uk.keep_div = P.p_uv.keep_div = -1;       // the tables are written once, here: the kernels need not wait for them
    }
    RC(dmalloc(A, &P.qkv_out, (size_t)R * QKVN));
    RC(dmalloc(A, &P.o_out, (size_t)R * H));
    RC(dmalloc(A, &P.gu_out, (size_t)R * 2 * Fmax));
    RC(dmalloc(A, &P.down_out, (size_t)R * H));
    RC(dmalloc(A, &P.ao_hi, (size_t)P.BN * QD));
    RC(dmalloc(A, &P.ao_lo, (size_t)P.BN * QD));
    RC(dmalloc(A, &P.ff_hi, (size_t)P.BN * Fmax));
    RC(dmalloc(A, &P.ff_lo, (size_t)P.BN * Fmax));
    if (e->mla && e->moe_E && e->first_dense > 0) {   // the dense feed-forward layers of a decoder with expert layers
      RC(gemm_plan_create(&P.p_gu_d, e->w0_gu_d, 2 * Fd, H, P.xn_hi, P.xn_lo, R, P.BN, P.gu_out, P.ws, e->num_sms));
      RC(gemm_plan_create(&P.p_down_d, e->w0_down_d, H, Fd, P.ff_hi, P.ff_lo, R, P.BN, P.down_out, P.ws, e->num_sms));
    }
    // the plans carry layer 0's weights; the per-layer tensor maps override them at launch
    RC(gemm_plan_create(&P.p_qkv, e->w0_qkv, QKVN, H, P.xn_hi, P.xn_lo, R, P.BN, P.qkv_out, P.ws, e->num_sms));
    RC(gemm_plan_create(&P.p_o, e->w0_o, H, QD, P.ao_hi, P.ao_lo, R, P.BN, P.o_out, P.ws, e->num_sms));
    // expert layers without groups: the routing weight and the SwiGLU in the epilogue of the GEMM over all experts'
    // gate / up rows (65..128 rows, where the grouped form below does not apply; up to 64 rows the masked store plus a
    // SwiGLU kernel measured faster: the epilogue would write zeros for every pair that was not selected)
    const bool moe_fused = fuse_swiglu && e->moe_E && P.BN > 64 && P.BN <= 128 &&
                           gemm_swiglu_blocks_half(e->moe_F, e->moe_E + e->moe_S, e->num_sms) > 0;
    if (fuse_swiglu && !e->moe_E && P.BN <= 128)
      RC(gemm_plan_create_swiglu(&P.p_gu, e->w0_gu, F, H, P.xn_hi, P.xn_lo, R, P.BN, P.ff_hi, P.ff_lo, e->num_sms));
    else if (!moe_fused)
      RC(gemm_plan_create(&P.p_gu, e->w0_gu, 2 * F, H, P.xn_hi, P.xn_lo, R, P.BN, P.gu_out, P.ws, e->num_sms));
    RC(gemm_plan_create(&P.p_down, e->w0_down, H, F, P.ff_hi, P.ff_lo, R, P.BN, P.down_out, P.ws, e->num_sms));
    if (e->moe_E) {
      const int NB = e->moe_E + e->moe_S;
      RC(dmalloc(A, &P.moe_w, (size_t)R * NB));
      if (moe_fused)
        RC(gemm_plan_create_swiglu_blocks(&P.p_gu, e->w0_gu, NB, e->moe_F, H, P.xn_hi, P.xn_lo, R, P.BN, P.ff_hi, P.ff_lo, P.moe_w,
                                          e->num_sms));
      else if ((2 * e->moe_F) % GEMM_TILE_N == 0) {   // a weight tile belongs to one expert: rows that did not
        P.p_gu.row_keep = P.moe_w;                  // select it are not stored (the SwiGLU does not read them)
        P.p_gu.keep_pitch = NB;
        P.p_gu.keep_div = 2 * e->moe_F / GEMM_TILE_N;
      }
      if (grouped && (2 * e->moe_F) % GEMM_TILE_N == 0 && H % GEMM_TILE_N == 0) {
        // prefill chunks: every row through every expert would be (E + S) / top_k times the MMA work, which a
        // chunk of 256 rows does pay for; the rows of an expert are gathered into blocks of 64 instead
        const int Fm = e->moe_F;
        MoeGroups &g = P.grp;
        g.n_groups_max = moe_max_groups(R, e->moe_E, e->moe_S, e->moe_K);
        const size_t slots = (size_t)g.n_groups_max * MOE_GROUP_ROWS;
        RC(dmalloc(A, &g.tab_up, (size_t)g.n_groups_max * 3 + 1));
        RC(dmalloc(A, &g.tab_down, (size_t)g.n_groups_max * 3 + 1));
        RC(dmalloc(A, &g.group_expert, (size_t)g.n_groups_max));
        RC(dmalloc(A, &g.slot_row, slots));
        RC(dmalloc(A, &g.slot_of, (size_t)R * NB));
        RC(dmalloc(A, &g.slot_w, slots));
        RC(dmalloc(A, &P.xg_hi, slots * H));
        RC(dmalloc(A, &P.xg_lo, slots * H));
        RC(dmalloc(A, &P.hg_hi, slots * Fm));
        RC(dmalloc(A, &P.hg_lo, slots * Fm));
        RC(dmalloc(A, &P.gug_out, slots * 2 * Fm));
        RC(dmalloc(A, &P.yg_out, slots * H));
        RC(dmalloc(A, &P.plain_tiles, (size_t)(H / GEMM_TILE_N + 1)));
        // gate / up per group with the routing weight and the SwiGLU in the epilogue where a tile width divides the
        // experts' width, else fp32 sums and a kernel of its own
        const int half = gemm_swiglu_blocks_half(Fm, NB, e->num_sms);
        if (half)
          RC(gemm_plan_create_grouped_swiglu(&P.p_gug, e->w0_gu, (long long)NB * 2 * Fm, Fm, H, half, P.xg_hi, P.xg_lo, g.n_groups_max,
                                             MOE_GROUP_ROWS, P.hg_hi, P.hg_lo, g.slot_w, g.tab_up, e->num_sms));
        else
          RC(gemm_plan_create_grouped(&P.p_gug, e->w0_gu, (long long)NB * 2 * Fm, H, 2 * Fm, H, P.xg_hi, P.xg_lo, g.n_groups_max,
                                      MOE_GROUP_ROWS, P.gug_out, g.tab_up, e->num_sms));
        RC(gemm_plan_create_grouped(&P.p_dng, e->w0_down, H, NB * Fm, H, Fm, P.hg_hi, P.hg_lo, g.n_groups_max, MOE_GROUP_ROWS,
                                    P.yg_out, g.tab_down, e->num_sms));
        P.grouped = true;
      }
    }
  }
  if (lm) {
    RC(dmalloc(A, &P.logits, (size_t)R * V));
    RC(gemm_plan_create(&P.p_lm, e->lm_head, V, H, P.xn_hi, P.xn_lo, R, P.BN, P.logits, P.ws, e->num_sms));
  }
  return CORUN_OK;
}

void program_destroy(Program &P) {
  gemm_plan_destroy(&P.p_qkv);
  gemm_plan_destroy(&P.p_o);
  gemm_plan_destroy(&P.p_gu);
  gemm_plan_destroy(&P.p_down);
  gemm_plan_destroy(&P.p_lm);
  gemm_plan_destroy(&P.p_gug);
  gemm_plan_destroy(&P.p_dng);
  gemm_plan_destroy(&P.p_uk);
  gemm_plan_destroy(&P.p_uv);
  gemm_plan_destroy(&P.p_gu_d);
  gemm_plan_destroy(&P.p_down_d);
  for (void *p : P.allocs) cudaFree(p);
  P.allocs.clear();
}

KvLayout kv_layout(const corun_engine *e) {
  return KvLayout{e->kv_pool, e->d_block_table, e->max_blocks, e->sh.n_kv_heads, e->sh.head_dim, e->layer_stride,
                  (long long)e->pool_blocks, e->B};
}

// The result of a layer's feed-forward part as the next kernel reads it: the down GEMM's partials, or (grouped
// Mixture-of-Experts form) the combined plain matrix.
bool dense_layer(const corun_engine *e, int layer) { return e->mla && e->moe_E && layer < e->first_dense; }

GemmOut ffn_out(const corun_engine *e, const Program &P, int layer) {
  if (dense_layer(e, layer)) return P.p_down_d.out();
  if (P.grouped) return GemmOut{P.down_out, nullptr, P.plain_tiles, P.plain_tiles, P.p_down.N, P.p_down.KB, P.BN};
  return P.p_down.out();
}

// Enqueues embed -> all layers (ends with the last down GEMM).  Counts launches.
int run_layers(corun_engine *e, Program &P, int *launches) {
  const corun_shape &s = e->sh;
  const Rows rows{P.row_token, P.row_pos, P.row_active, P.row_slot, P.R};
  const KvLayout kv = kv_layout(e);
  int n = 0;
  if (&P == &e->dec && !e->mla) {                   // the prefill attention kernel needs no item list
    CK(launch_attn_worklist(rows, e->sh.n_kv_heads, P.att_work, P.att_n_work, P.att_pool, s.n_layers, e->whole_pairs, e->st));   // the same items serve every layer
    n += 1;
  }
  // (debug) slice of the step trace for the idx-th GEMM of the decode program: [num_sms][8] stamps
  auto tr = [&](int idx) -> unsigned long long * {
    return (e->step_trace && &P == &e->dec) ? e->step_trace + (size_t)idx * e->num_sms * 8 : nullptr;
  };
  int stage = 0;
  const int stop = (e->eager && &P == &e->dec) ? e->stop_after : -1;
#define STAGE(call)                                   \
  do {                                                \
    if (stop >= 0 && stage >= stop) return CORUN_OK;  \
    CK(call);                                         \
    ++stage;                                          \
  } while (0)
  for (int l = 0; l < s.n_layers; ++l) {
    GemmOut prev = ffn_out(e, P, l > 0 ? l - 1 : 0);
    STAGE(launch_resid_norm(P.h, s.hidden, e->embed, rows, l == 0 ? nullptr : &prev, e->attn_norm[l], s.rms_eps,
                            P.xn_hi, P.xn_lo, e->st));
    STAGE(gemm_launch(P.p_qkv, &e->tm_qkv[l], e->d_status, e->st, tr(4 * l + 0), true));
    if (e->mla) {
      // cache append and query parts -> q_lat = W_uk^T q_nope per head -> absorbed attention over the row's latent
      // pages (decode rows and prefill rows alike) -> [. | o] = W_kv_b o_lat per head -> the value part, split
      const MlaDims &md = e->md;
      const MlaCache cache{e->kv_pool + (size_t)l * e->layer_stride, e->d_block_table, e->max_blocks, e->B, (long long)e->pool_blocks, e->kv_run};
      STAGE(launch_mla_post(P.p_qkv.out(), rows, e->d_rope, md, e->kv_norm[l], s.rms_eps, cache, P.RPH, P.qn_hi, P.qn_lo, P.q_rope,
                            e->d_status, e->st));
      STAGE(gemm_launch(P.p_uk, &e->tm_uk[l], e->d_status, e->st, nullptr, true));
      STAGE(launch_mla_attention(e->tm_c[l], e->tm_cv[l], P.q_lat, md.rank, (long long)P.RPH * md.rank, P.q_rope, e->d_block_table,
                                 e->max_blocks, nullptr, &rows, P.R, md, 1.0f / sqrtf((float)(md.nope + md.rope)), e->mla_splits,
                                 P.mla_ml, P.mla_po, nullptr, P.ol_hi, P.ol_lo, P.RPH, e->num_sms, e->d_status, true, e->st, e->kv_run));
      STAGE(gemm_launch(P.p_uv, &e->tm_uv[l], e->d_status, e->st, nullptr, true));
      STAGE(launch_mla_ao_split(P.uv_out, P.R, P.RPH, md, P.ao_hi, P.ao_lo, e->st));
      n += 3 + (&P == &e->dec ? 0 : 1);               // beyond the count below: two grouped GEMMs, the split, and in prefill too a second attention kernel
    } else {
    STAGE(launch_qkv_post(P.p_qkv.out(), rows, e->d_rope, s.n_q_heads, kv, l, P.q, e->d_status, e->st));
    // (the decode kernel takes the one-box-per-tile view of the pages, the prefill kernel the row view)
    STAGE(launch_attention(&P == &e->dec ? e->tm_k4[l] : e->tm_k[l], &P == &e->dec ? e->tm_k4[l] : e->tm_v[l], P.q, rows, s.n_q_heads, kv, l, e->max_splits, P.att_work, P.att_n_work,
                           e->num_sms, P.part_acc, P.part_ml, P.att_pool + l, P.ao_hi, P.ao_lo, &P == &e->dec ? (e->whole_pairs ? 2 : 0) : 1,
                           e->d_status, e->st));
    }
    STAGE(gemm_launch(P.p_o, &e->tm_o[l], e->d_status, e->st, tr(4 * l + 1), true));
    GemmOut o = P.p_o.out();
    STAGE(launch_resid_norm(P.h, s.hidden, nullptr, rows, &o, e->mlp_norm[l], s.rms_eps, P.xn_hi, P.xn_lo, e->st));
    if (dense_layer(e, l)) {
      STAGE(gemm_launch(P.p_gu_d, &e->tm_gu_d[l], e->d_status, e->st, nullptr, true));
      STAGE(launch_swiglu(P.p_gu_d.out(), P.R, e->dense_ffn, P.ff_hi, P.ff_lo, e->st));
      STAGE(gemm_launch(P.p_down_d, &e->tm_down_d[l], e->d_status, e->st, nullptr, true));
      n += 9 + (&P == &e->dec ? 1 : 0);
      continue;
    } else if (e->moe_E && P.grouped) {
      // router -> top-k weights -> rows grouped by expert -> gate / up, SwiGLU and down per group -> the row's
      // experts summed in ascending expert id
      const int NB = e->moe_E + e->moe_S;
      STAGE(launch_moe_router(P.xn_hi, P.xn_lo, s.hidden, e->router[l], P.R, e->moe_E, e->moe_S, e->moe_K, e->moe_renorm, P.moe_w, nullptr,
                              nullptr, e->st));
      STAGE(launch_moe_group(P.moe_w, P.row_active, P.R, e->moe_E, e->moe_S, e->moe_F, P.grp, e->st));
      STAGE(launch_moe_gather(P.xn_hi, P.xn_lo, s.hidden, P.grp, P.xg_hi, P.xg_lo, e->st));
      if (P.p_gug.sw_hi) {                            // routing weight and SwiGLU in the GEMM's epilogue
        STAGE(gemm_launch(P.p_gug, &e->tm_gu_half[l], e->d_status, e->st, nullptr, true));
        n -= 1;
      } else {
        STAGE(gemm_launch(P.p_gug, &e->tm_gu[l], e->d_status, e->st, nullptr, true));
        STAGE(launch_moe_swiglu_grouped(P.gug_out, P.moe_w, NB, e->moe_F, P.grp, P.hg_hi, P.hg_lo, e->st));
      }
      STAGE(gemm_launch(P.p_dng, &e->tm_down[l], e->d_status, e->st, nullptr, true));
      STAGE(launch_moe_combine(P.yg_out, P.row_active, P.R, NB, s.hidden, P.grp, P.down_out, e->st));
      n += 13 + (&P == &e->dec ? 1 : 0);
      continue;
    } else if (e->moe_E) {
      // router -> top-k weights -> all experts' gate / up (rows that did not select a tile's expert are not
      // stored) -> masked, weighted SwiGLU; the down GEMM then sums over the row's experts in its accumulator
      STAGE(launch_moe_router(P.xn_hi, P.xn_lo, s.hidden, e->router[l], P.R, e->moe_E, e->moe_S, e->moe_K, e->moe_renorm, P.moe_w, nullptr,
                              nullptr, e->st));
      if (P.p_gu.sw_hi) {                             // routing weight and SwiGLU in the GEMM's epilogue
        STAGE(gemm_launch(P.p_gu, &e->tm_gu_half[l], e->d_status, e->st, tr(4 * l + 2), true));
      } else {                                        // (the router is the one kernel beyond the count below)
        STAGE(gemm_launch(P.p_gu, &e->tm_gu[l], e->d_status, e->st, tr(4 * l + 2), true));
        STAGE(launch_moe_swiglu(P.p_gu.out(), P.moe_w, P.R, e->moe_F, e->moe_E + e->moe_S, P.ff_hi, P.ff_lo, e->st));
        n += 1;
      }
    } else {
      if (P.p_gu.sw_hi) {                             // SwiGLU in the GEMM's epilogue
        STAGE(gemm_launch(P.p_gu, &e->tm_gu_half[l], e->d_status, e->st, tr(4 * l + 2), true));
        n -= 1;
      } else {
        STAGE(gemm_launch(P.p_gu, &e->tm_gu[l], e->d_status, e->st, tr(4 * l + 2), true));
        STAGE(launch_swiglu(P.p_gu.out(), P.R, s.ffn, P.ff_hi, P.ff_lo, e->st));
      }
    }
    STAGE(gemm_launch(P.p_down, &e->tm_down[l], e->d_status, e->st, tr(4 * l + 3), true));
    n += 9 + (&P == &e->dec ? 1 : 0);   // decode attention is two kernels (splits, combine)
  }
#undef STAGE
  if (launches) *launches += n;
  return CORUN_OK;
}

// One decode iteration on the stream (what the graph captures).
int enqueue_decode_body(corun_engine *e, int *launches) {
  Program &P = e->dec;
  const corun_shape &s = e->sh;
  int n = 0;
  // mask and seeds are read from the pinned staging buffers by the first kernel, tokens and status are written to
  // them by the last one (zero-copy): a copy node in a graph costs several microseconds, these are 836 bytes
  CK(launch_prepare_rows(e->h_active, e->h_seeds, e->d_seeds, e->d_in_use, e->d_ctx, e->d_pending, e->d_temp, e->d_top_p, e->d_step, e->B,
                         P.row_token, P.row_pos, P.row_active, P.row_slot, P.do_sample, P.row_temp, P.row_top_p, P.row_step, P.slot_row,
                         P.row_blocks, e->st));
  n += 1;
  RC(run_layers(e, P, &n));
  if (!(e->eager && e->stop_after >= 0)) {   // (debug) a truncated layer stack skips the tail too
    const Rows rows{P.row_token, P.row_pos, P.row_active, P.row_slot, P.R};
    GemmOut prev = ffn_out(e, P, s.n_layers - 1);
    CK(launch_resid_norm(P.h, s.hidden, nullptr, rows, &prev, e->final_norm, s.rms_eps, P.xn_hi, P.xn_lo, e->st));
    CK(gemm_launch(P.p_lm, nullptr, e->d_status, e->st, nullptr, true));
    CK(gemm_fixup_launch(P.p_lm, e->st, true));
    SampleArgs sa{P.logits, s.vocab, P.do_sample, P.row_temp, P.row_top_p, e->d_seeds, P.row_step, nullptr, P.sampled};   // all by row
    CK(launch_sampler(sa, P.R, e->st, true));
    CK(launch_advance(P.slot_row, P.row_active, P.sampled, e->B, e->d_ctx, e->d_step, e->d_pending, e->h_out_tokens, e->d_status, e->h_status,
                      e->st));
    n += 4 + (P.p_lm.n_split_tiles ? 1 : 0);
  }
  if (e->eager && e->stop_after >= 0)            // (debug) no last kernel ran: fetch the status word the plain way
    CK(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, e->st));
  if (launches) *launches = n;
  return CORUN_OK;
}

int check_status(corun_engine *e) {
  if (*e->h_status == 4) return CORUN_EINVAL;   // DEV_BAD_INDEX: an index check of a -DCORUN_CHECKED build failed
  if (*e->h_status != 0) return CORUN_ETIMEOUT;
  return CORUN_OK;
}

int sync_stream(corun_engine *e) {
  CK(cudaStreamSynchronize(e->st));
  e->in_flight = false;
  return CORUN_OK;
}

int reserve_blocks(corun_engine *e, int slot, int reserve_len) {
  const int run_tokens = KV_BLOCK * e->kv_run;
  const int need = (reserve_len + run_tokens - 1) / run_tokens;   // runs
  if ((size_t)need > e->free_blocks.size()) return CORUN_ENOSPACE;
  std::vector<int> &mine = e->slot_blocks[slot];
  mine.clear();
  std::vector<int> row(e->max_blocks, 0);
  for (int i = 0; i < need; ++i) {
    mine.push_back(e->free_blocks.back());
    e->free_blocks.pop_back();
    for (int j = 0; j < e->kv_run && i * e->kv_run + j < e->max_blocks; ++j) row[i * e->kv_run + j] = mine.back() * e->kv_run + j;
  }
  CK(cudaMemcpyAsync(e->d_block_table + (size_t)slot * e->max_blocks, row.data(), e->max_blocks * sizeof(int),
                     cudaMemcpyHostToDevice, e->st));
  CK(cudaStreamSynchronize(e->st));   // `row` is pageable and local
  return CORUN_OK;
}

int set_slot_state(corun_engine *e, int slot, int in_use, int ctx, int step, int pending, float temp, float top_p) {
  CK(cudaMemcpyAsync(e->d_in_use + slot, &in_use, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_ctx + slot, &ctx, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_step + slot, &step, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_pending + slot, &pending, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_temp + slot, &temp, sizeof(float), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_top_p + slot, &top_p, sizeof(float), cudaMemcpyHostToDevice, e->st));
  CK(cudaStreamSynchronize(e->st));
  return CORUN_OK;
}

bool slot_ok(const corun_engine *e, int slot) { return slot >= 0 && slot < e->B; }

}  // namespace

extern "C" {

int corun_last_cuda_error(void) { return g_last_cuda_error; }

const char *corun_strerror(int st) {
  switch (st) {
    case CORUN_OK: return "ok";
    case CORUN_EINVAL: return "invalid argument";
    case CORUN_ESLOT: return "bad slot (out of range, busy, or empty)";
    case CORUN_ENOSPACE: return "KV pool cannot hold the reserved sequence";
    case CORUN_ECTX: return "an active slot is at its reserved length";
    case CORUN_ECUDA: return "CUDA error";
    case CORUN_ETIMEOUT: return "a bounded device-side wait expired";
    case CORUN_ENOMEM: return "out of memory";
    case CORUN_ELIMIT: return "size exceeds the fixed capacity of corun_gemm_static";
    default: return "unknown status";
  }
}

static int engine_create(const corun_shape *shape, const corun_weights *w, const corun_moe_layers *moe,
                         const corun_mla_layers *mla, int32_t B, int32_t max_context, int32_t kv_block,
                         int64_t kv_pool_blocks, void *cuda_stream, corun_engine **out) {
  if (!shape || !w || !out) return CORUN_EINVAL;
  *out = nullptr;
  corun_shape s = *shape;
  if (s.n_layers < 1) return CORUN_EINVAL;
  int first_dense = 0, dense_ffn = 0;                // MLA: layers with a dense feed-forward, and its width
  if (mla) {
    if (s.arch != 0 && s.arch != 1) return CORUN_EINVAL;
    s.arch = 0;
    if ((mla->kv_lora_rank != 256 && mla->kv_lora_rank != 512) || mla->qk_nope < 64 || mla->qk_nope % 64 || mla->qk_rope < 8 ||
        mla->qk_rope > 64 || mla->qk_rope % 8 || mla->v_head < 64 || (mla->qk_nope + mla->v_head) % 256 || s.n_q_heads < 1 ||
        s.n_q_heads > 16 || mla->first_dense < 0 || mla->first_dense > s.n_layers || (!moe && mla->first_dense != s.n_layers) ||
        !mla->kv_norm || !mla->wkv_b)
      return CORUN_EINVAL;
    for (int l = 0; l < s.n_layers; ++l)
      if (!mla->kv_norm[l] || !mla->wkv_b[l]) return CORUN_EINVAL;
    first_dense = mla->first_dense;
    dense_ffn = s.ffn;
    if (first_dense > 0 && (dense_ffn < 64 || dense_ffn % 64 || !w->wgate_up || !w->wdown)) return CORUN_EINVAL;
    for (int l = 0; l < first_dense; ++l)
      if (!w->wgate_up[l] || !w->wdown[l]) return CORUN_EINVAL;
    if (first_dense == s.n_layers) moe = nullptr;   // no expert layer at all
    s.head_dim = mla->v_head;                        // the o-projection's K is n_q_heads * v_head
    s.n_kv_heads = s.n_q_heads;
  }
  if (moe) {
    if (moe->n_experts < 1 || moe->n_experts > 256 || moe->top_k < 1 || moe->top_k > 16 || moe->top_k > moe->n_experts ||
        moe->expert_ffn < 64 || moe->expert_ffn % 64 || moe->n_shared < 0 || !moe->router || !moe->gate_up || !moe->down)
      return CORUN_EINVAL;
    for (int l = first_dense; l < s.n_layers; ++l)
      if (!moe->router[l] || !moe->gate_up[l] || !moe->down[l]) return CORUN_EINVAL;
    s.ffn = (moe->n_experts + moe->n_shared) * moe->expert_ffn;   // the feed-forward width the row program sees
  }
  if (s.arch != 0 || s.n_layers < 1 || s.hidden < 64 || s.hidden % 64 || s.ffn < 64 || s.ffn % 64 || s.vocab < 1)
    return CORUN_EINVAL;
  if (!mla && s.head_dim != 64 && s.head_dim != 128) return CORUN_EINVAL;
  if (s.n_q_heads < 1 || s.n_kv_heads < 1 || s.n_q_heads % s.n_kv_heads) return CORUN_EINVAL;
  const int group = s.n_q_heads / s.n_kv_heads;
  if (group != 1 && group != 2 && group != 4 && group != 8) return CORUN_EINVAL;
  if ((s.n_q_heads * s.head_dim) % 64) return CORUN_EINVAL;
  if (!(s.rms_eps >= 0.f) || !(s.rope_theta > 0.f)) return CORUN_EINVAL;
  // kv_block: 16, or (latent caches only) 64: pages of 16 tokens handed out in aligned runs of four
  if (B < 1 || B > 256 || max_context < 1 || max_context > 256 * ATT_SPLIT || !(kv_block == KV_BLOCK || (mla && kv_block == 4 * KV_BLOCK)) ||
      kv_pool_blocks < 0)
    return CORUN_EINVAL;
  if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wqkv || !w->wo || !w->mlp_norm ||
      (!moe && (!w->wgate_up || !w->wdown)))
    return CORUN_EINVAL;
  for (int l = 0; l < s.n_layers; ++l)
    if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->mlp_norm[l] || (!moe && (!w->wgate_up[l] || !w->wdown[l])))
      return CORUN_EINVAL;
  const int Lm = moe ? first_dense : 0;              // the first layer with experts (whose weights the plans are made on)

  int dev = 0;
  CK(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CK(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return CORUN_ECUDA;   // tcgen05 / TMEM kernels: sm_100a only

  corun_engine *e = new (std::nothrow) corun_engine();
  if (!e) return CORUN_ENOMEM;
  auto fail = [&](int rc) {
    corun_destroy(e);
    return rc;
  };
  e->sh = s;
  e->B = B;
  e->max_ctx = max_context;
  e->kv_run = kv_block / KV_BLOCK;
  e->max_blocks = (max_context + kv_block - 1) / kv_block * e->kv_run;   // pages of 16 tokens, whole runs
  e->max_splits = (max_context + ATT_SPLIT - 1) / ATT_SPLIT;
  e->num_sms = prop.multiProcessorCount;
  e->st = (cudaStream_t)cuda_stream;
  if (!e->st) {   // the legacy default stream cannot be captured: use a private one
    if (cudaStreamCreateWithFlags(&e->st, cudaStreamNonBlocking) != cudaSuccess) return fail(CORUN_ECUDA);
    e->own_stream = true;
  }
  e->w0_qkv = w->wqkv[0];
  e->w0_o = w->wo[0];
  e->w0_gu = moe ? moe->gate_up[Lm] : w->wgate_up[0];
  e->w0_down = moe ? moe->down[Lm] : w->wdown[0];
  if (mla) {
    e->mla = true;
    e->md = MlaDims{s.n_q_heads, mla->kv_lora_rank, mla->qk_nope, mla->qk_rope, mla->v_head};
    e->first_dense = first_dense;
    e->dense_ffn = moe ? dense_ffn : 0;
    e->mla_splits = mla_max_splits(max_context);
    e->w0_uv = mla->wkv_b[0];
    if (moe && first_dense > 0) { e->w0_gu_d = w->wgate_up[0]; e->w0_down_d = w->wdown[0]; }
  }
  if (moe) {
    e->moe_E = moe->n_experts;
    e->moe_K = moe->top_k;
    e->moe_F = moe->expert_ffn;
    e->moe_S = moe->n_shared;
    e->moe_renorm = moe->renormalize ? 1 : 0;
  }
  e->pool_blocks = kv_pool_blocks ? kv_pool_blocks * e->kv_run : (int64_t)B * e->max_blocks;   // in pages of 16 tokens
  if (!kv_pool_blocks) {
    // default size: a full reservation for every slot, or as many pages as fit beside 6 GiB that are
    // left for the programs' buffers, whichever is less (admission then refuses what does not fit)
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) return fail(CORUN_ECUDA);
    const size_t page_b = mla ? (size_t)s.n_layers * KV_BLOCK * (size_t)mla_token_halfs(mla->kv_lora_rank + mla->qk_rope, e->kv_run) * sizeof(__half)
                              : (size_t)s.n_layers * 2 * s.n_kv_heads * KV_BLOCK * s.head_dim * sizeof(__half);
    const size_t keep = (size_t)6 << 30;
    const int64_t fit = free_b > keep ? (int64_t)((free_b - keep) / page_b) : 0;
    if (fit < e->pool_blocks) e->pool_blocks = fit / e->kv_run * e->kv_run;
    if (e->pool_blocks < e->kv_run) return fail(CORUN_ENOMEM);
  }
  e->chunk = 256;
  if (const char *c = getenv("CORUN_ATTN_WHOLE_PAIRS")) e->whole_pairs = atoi(c) != 0;   // ablation only
  if (const char *c = getenv("CORUN_PREFILL_CHUNK")) {
    const int v = atoi(c);
    if (v >= 16 && v <= 256 && v % 16 == 0) e->chunk = v;
  }
  e->embed = (const bf16 *)w->embed;
  e->lm_head = (const bf16 *)w->lm_head;
  e->final_norm = (const bf16 *)w->final_norm;
  const int H = s.hidden, QD = s.n_q_heads * s.head_dim, KD = s.n_kv_heads * s.head_dim, F = s.ffn;
  e->tm_qkv.resize(s.n_layers);
  e->tm_o.resize(s.n_layers);
  e->tm_gu.resize(s.n_layers);
  e->tm_down.resize(s.n_layers);
  const int moe_half = moe ? gemm_swiglu_blocks_half(moe->expert_ffn, moe->n_experts + moe->n_shared, e->num_sms) : 0;
  if (!moe || moe_half) e->tm_gu_half.resize(s.n_layers);
  for (int l = 0; l < s.n_layers; ++l) {
    e->attn_norm.push_back((const bf16 *)w->attn_norm[l]);
    e->mlp_norm.push_back((const bf16 *)w->mlp_norm[l]);
    int rc;
    const int qkv_rows = mla ? s.n_q_heads * (mla->qk_nope + mla->qk_rope) + mla->kv_lora_rank + mla->qk_rope : QD + 2 * KD;
    if ((rc = gemm_encode_map(&e->tm_qkv[l], w->wqkv[l], qkv_rows, H, GEMM_TILE_N))) return fail(rc);
    if ((rc = gemm_encode_map(&e->tm_o[l], w->wo[l], H, QD, GEMM_TILE_N))) return fail(rc);
    if (moe && l < first_dense) {                   // a dense feed-forward layer of a decoder with expert layers
      if (e->tm_gu_d.empty()) { e->tm_gu_d.resize(s.n_layers); e->tm_down_d.resize(s.n_layers); }
      if ((rc = gemm_encode_map(&e->tm_gu_d[l], w->wgate_up[l], 2 * dense_ffn, H, GEMM_TILE_N))) return fail(rc);
      if ((rc = gemm_encode_map(&e->tm_down_d[l], w->wdown[l], H, dense_ffn, GEMM_TILE_N))) return fail(rc);
      continue;
    }
    if ((rc = gemm_encode_map(&e->tm_gu[l], moe ? moe->gate_up[l] : w->wgate_up[l], 2 * F, H, GEMM_TILE_N))) return fail(rc);
    if ((rc = gemm_encode_map(&e->tm_down[l], moe ? moe->down[l] : w->wdown[l], H, F, GEMM_TILE_N))) return fail(rc);
    if (!moe && (rc = gemm_encode_map(&e->tm_gu_half[l], w->wgate_up[l], 2 * F, H, gemm_swiglu_half(F, e->num_sms)))) return fail(rc);
    if (moe && moe_half && (rc = gemm_encode_map(&e->tm_gu_half[l], moe->gate_up[l], 2 * F, H, moe_half))) return fail(rc);
  }
  if (mla) {
    // the key up-projections transposed (q_lat = W_uk^T q_nope is a GEMM over rows of W_uk^T), and per layer
    // the maps of the two grouped up-projection GEMMs
    int rc;
    const MlaDims &md = e->md;
    const size_t per_layer = (size_t)md.nh * md.rank * md.nope;
    if ((rc = dmalloc(e->allocs, &e->w_ukT, per_layer * s.n_layers, false))) return fail(rc);
    e->tm_uk.resize(s.n_layers);
    e->tm_uv.resize(s.n_layers);
    for (int l = 0; l < s.n_layers; ++l) {
      e->kv_norm.push_back((const bf16 *)mla->kv_norm[l]);
      bf16 *dst = e->w_ukT + (size_t)l * per_layer;
      if (launch_mla_transpose_uk((const bf16 *)mla->wkv_b[l], md, dst, 0) != cudaSuccess) return fail(CORUN_ECUDA);
      if ((rc = gemm_encode_map(&e->tm_uk[l], dst, md.nh * md.rank, md.nope, GEMM_TILE_N))) return fail(rc);
      if ((rc = gemm_encode_map(&e->tm_uv[l], mla->wkv_b[l], md.nh * (md.nope + md.vh), md.rank, GEMM_TILE_N))) return fail(rc);
    }
  }
  if (moe) {
    if (H > 12288) return fail(CORUN_EINVAL);       // the router kernel keeps a row in shared memory
    for (int l = 0; l < s.n_layers; ++l) {
      if (l >= first_dense && ((uintptr_t)moe->router[l] & 15u)) return fail(CORUN_EINVAL);
      e->router.push_back(l >= first_dense ? (const bf16 *)moe->router[l] : nullptr);
    }
  }

  auto &A = e->allocs;
  int rc;
  e->layer_stride = mla ? (size_t)e->pool_blocks * KV_BLOCK * (size_t)mla_token_halfs(e->md.rank + e->md.rope, e->kv_run)
                        : (size_t)e->pool_blocks * 2 * s.n_kv_heads * KV_BLOCK * s.head_dim;
  // zero-filled: masked positions of a page are multiplied by zero weights, so they must be finite
  if ((rc = dmalloc(A, &e->kv_pool, e->layer_stride * s.n_layers, true))) return fail(rc);
  if (mla) {
    // one layer's pages: rows of rank + rope halfs, 16 per page
    e->tm_c.resize(s.n_layers);
    e->tm_cv.resize(s.n_layers);
    for (int l = 0; l < s.n_layers; ++l)
      if ((rc = mla_encode_maps(&e->tm_c[l], &e->tm_cv[l], e->kv_pool + (size_t)l * e->layer_stride, e->pool_blocks, e->md.rank, e->md.rope,
                                e->kv_run)))
        return fail(rc);
  } else {
    // one layer's pages seen as rows of hd halfs (16 rows per page and head, keys first, then values)
    const unsigned long long halfs = (unsigned long long)e->layer_stride;
    if (halfs / KV_BLOCK >= (1ull << 31)) return fail(CORUN_EINVAL);
    e->tm_k.resize(s.n_layers);
    e->tm_v.resize(s.n_layers);
    for (int l = 0; l < s.n_layers; ++l) {
      const __half *base = e->kv_pool + (size_t)l * e->layer_stride;
      if ((rc = tma_encode_2d(&e->tm_k[l], base, 1, halfs / s.head_dim, s.head_dim, KV_BLOCK, 64))) return fail(rc);
      e->tm_v[l] = e->tm_k[l];   // keys and values are cached alike: the same view serves both
      // decode attention: a tile's 16 tokens x head_dim in ONE box, [2 groups of 8 tokens][halves of 64 dims][8][64]
      const unsigned long long row_b = (unsigned long long)s.head_dim * 2;
      const unsigned long long d4[4] = {64, 8, (unsigned long long)(s.head_dim / 64), halfs / s.head_dim / 8};
      const unsigned long long s4[3] = {row_b, 128, 8 * row_b};
      const unsigned b4[4] = {64, 8, (unsigned)(s.head_dim / 64), 2};
      e->tm_k4.emplace_back();
      if ((rc = tma_encode_fp16_4d(&e->tm_k4[l], base, d4, s4, b4))) return fail(rc);
    }
    if (attention_prepare() != cudaSuccess) return fail(CORUN_ECUDA);
  }
  if ((rc = dmalloc(A, &e->d_block_table, (size_t)B * e->max_blocks))) return fail(rc);
  if ((rc = dmalloc(A, &e->d_in_use, B)) || (rc = dmalloc(A, &e->d_ctx, B)) || (rc = dmalloc(A, &e->d_step, B)) ||
      (rc = dmalloc(A, &e->d_pending, B)) || (rc = dmalloc(A, &e->d_temp, B)) || (rc = dmalloc(A, &e->d_top_p, B)) ||
      (rc = dmalloc(A, &e->d_seeds, B)) || (rc = dmalloc(A, &e->d_active, B)) || (rc = dmalloc(A, &e->d_out_tokens, B)) ||
      (rc = dmalloc(A, &e->d_status, 1)) || (rc = dmalloc(A, &e->d_pf_temp, 1)) || (rc = dmalloc(A, &e->d_pf_top_p, 1)) ||
      (rc = dmalloc(A, &e->d_pf_seed, 1)) || (rc = dmalloc(A, &e->d_pf_step, 1)) || (rc = dmalloc(A, &e->d_pf_one, 1)) ||
      (rc = dmalloc(A, &e->d_pf_tok, 1)) || (rc = dmalloc(A, &e->pf_logits, (size_t)B * s.vocab)))
    return fail(rc);
  e->logits_row.assign((size_t)B, -1);
  {
    // cos/sin of pos * theta^(-2i/hd), evaluated in fp64 on the host (hd: the rotated width)
    const int rot = mla ? mla->qk_rope : s.head_dim, half = rot / 2;
    std::vector<float2> tab((size_t)max_context * half);
    for (int p = 0; p < max_context; ++p)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)p * std::pow((double)s.rope_theta, -2.0 * (double)i / (double)rot);
        tab[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    if ((rc = dmalloc(A, &e->d_rope, tab.size(), false))) return fail(rc);
    if (cudaMemcpy(e->d_rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(CORUN_ECUDA);
    const int one = 1;
    if (cudaMemcpy(e->d_pf_one, &one, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return fail(CORUN_ECUDA);
  }
  const int64_t n_runs = e->pool_blocks / e->kv_run;
  e->free_blocks.resize((size_t)n_runs);
  for (int64_t i = 0; i < n_runs; ++i) e->free_blocks[(size_t)i] = (int)(n_runs - 1 - i);
  e->slot_blocks.resize(B);
  e->in_use.assign(B, 0);
  e->ctx.assign(B, 0);
  e->reserve.assign(B, 0);
  e->step.assign(B, 0);
  if (cudaMallocHost(&e->h_active, B) != cudaSuccess || cudaMallocHost(&e->h_seeds, B * sizeof(uint64_t)) != cudaSuccess ||
      cudaMallocHost(&e->h_out_tokens, B * sizeof(int)) != cudaSuccess ||
      cudaMallocHost(&e->h_status, sizeof(int)) != cudaSuccess ||
      cudaMallocHost(&e->h_rows, (size_t)5 * e->chunk * sizeof(int)) != cudaSuccess)
    return fail(CORUN_ENOMEM);
  memset(e->h_active, 0, B);
  memset(e->h_seeds, 0, B * sizeof(uint64_t));
  *e->h_status = 0;

#ifdef CORUN_BUILD_DEBUG
  if (const char *ts = getenv("CORUN_TRACE_STEP")) {
    if (atoi(ts) != 0 && (rc = dmalloc(A, &e->step_trace, (size_t)4 * s.n_layers * e->num_sms * 8))) return fail(rc);
  }
#endif
  // expert layers of the decode program: above 64 padded rows the grouped form (an expert's rows gathered into blocks of
  // 64: one MMA per k-slice covers the hi and lo halves of a block, where every row through every expert costs two on
  // 128 rows and keeps the tensor pipe as busy as the weight stream); up to 64 rows every row through every expert
  const bool dec_grouped = e->moe_E > 0 && pad16(B) > 64 && !getenv("CORUN_MOE_DECODE_DENSE");
  if ((rc = program_create(e, e->dec, B, true, true, dec_grouped, true))) return fail(rc);
  // the decode step's first kernel says which blocks of rows hold a request (64 rows each up to 128 padded rows, 128
  // rows each above); the GEMMs leave the others out (the one-row program has one block)
  for (GemmPlan *pl : {&e->dec.p_qkv, &e->dec.p_o, &e->dec.p_gu, &e->dec.p_down, &e->dec.p_lm, &e->dec.p_gu_d, &e->dec.p_down_d})
    pl->row_blocks = e->dec.row_blocks;
  if ((rc = program_create(e, e->pre, e->chunk, true, false, e->moe_E > 0 && !getenv("CORUN_MOE_PREFILL_DENSE")))) return fail(rc);
  // a prefill chunk is filled from row 0: the host says which blocks of rows it reaches (prefill_run)
  for (GemmPlan *pl : {&e->pre.p_qkv, &e->pre.p_o, &e->pre.p_gu, &e->pre.p_down, &e->pre.p_gu_d, &e->pre.p_down_d})
    pl->row_blocks = e->pre.row_blocks;
  if ((rc = program_create(e, e->lm1, 1, false, true))) return fail(rc);

  // the allocations above were cleared and filled through the legacy stream, which the engine's
  // stream does not wait for: drain the device once before the first launch
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(CORUN_ECUDA);
  // eager warm-up on an all-padding batch (also validates every launch), then capture
  if ((rc = enqueue_decode_body(e, &e->decode_launches))) return fail(rc);
  if (cudaStreamSynchronize(e->st) != cudaSuccess) return fail(CORUN_ECUDA);
  if ((rc = check_status(e))) return fail(rc);
  if (cudaStreamBeginCapture(e->st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return fail(CORUN_ECUDA);
  rc = enqueue_decode_body(e, nullptr);
  cudaError_t ce = cudaStreamEndCapture(e->st, &e->graph);
  if (rc) return fail(rc);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return fail(CORUN_ECUDA); }
  ce = cudaGraphInstantiate(&e->graph_exec, e->graph, 0);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return fail(CORUN_ECUDA); }
  *out = e;
  return CORUN_OK;
}

int corun_init(const corun_shape *shape, const corun_weights *w, int32_t B, int32_t max_context, int32_t kv_block,
               int64_t kv_pool_blocks, void *cuda_stream, corun_engine **out) {
  return engine_create(shape, w, nullptr, nullptr, B, max_context, kv_block, kv_pool_blocks, cuda_stream, out);
}

int corun_init_moe(const corun_shape *shape, const corun_weights *w, const corun_moe_layers *moe, int32_t B,
                   int32_t max_context, int32_t kv_block, int64_t kv_pool_blocks, void *cuda_stream, corun_engine **out) {
  if (!moe) return CORUN_EINVAL;
  return engine_create(shape, w, moe, nullptr, B, max_context, kv_block, kv_pool_blocks, cuda_stream, out);
}

int corun_init_mla(const corun_shape *shape, const corun_weights *w, const corun_mla_layers *mla, const corun_moe_layers *moe,
                   int32_t B, int32_t max_context, int32_t kv_block, int64_t kv_pool_blocks, void *cuda_stream,
                   corun_engine **out) {
  if (!mla) return CORUN_EINVAL;
  return engine_create(shape, w, moe, mla, B, max_context, kv_block, kv_pool_blocks, cuda_stream, out);
}

void corun_destroy(corun_engine *e) {
  if (!e) return;
  cudaStreamSynchronize(e->st);
  if (e->graph_exec) cudaGraphExecDestroy(e->graph_exec);
  if (e->graph) cudaGraphDestroy(e->graph);
  program_destroy(e->dec);
  program_destroy(e->pre);
  program_destroy(e->lm1);
  for (void *p : e->allocs) cudaFree(p);
  if (e->h_active) cudaFreeHost(e->h_active);
  if (e->h_seeds) cudaFreeHost(e->h_seeds);
  if (e->h_out_tokens) cudaFreeHost(e->h_out_tokens);
  if (e->h_status) cudaFreeHost(e->h_status);
  if (e->h_rows) cudaFreeHost(e->h_rows);
  if (e->own_stream) cudaStreamDestroy(e->st);
  delete e;
}

}  // extern "C"

namespace {

struct PfReq {
  int slot;
  const int32_t *tokens;
  int n, reserve;
  corun_sampling smp;
  uint64_t seed;
  int first;
};

// Final norm -> LM head (one row) -> sample with R(seed, 0) for the request whose last prompt token is row
// `row` of the chunk that has just run; the logits go to the slot's place among the prefill logits.
int prefill_finish_row(corun_engine *e, int row, PfReq &r) {
  const corun_shape &s = e->sh;
  Program &P = e->pre, &L = e->lm1;
  GemmOut prev = ffn_out(e, P, s.n_layers - 1);
  prev.direct += (size_t)row * prev.N;
  if (prev.ws) prev.ws += (size_t)row * GEMM_TILE_N;
  const Rows one{P.row_token + row, P.row_pos + row, P.row_active + row, P.row_slot + row, 1};
  CK(launch_resid_norm(P.h + (size_t)row * s.hidden, s.hidden, nullptr, one, &prev, e->final_norm, s.rms_eps, L.xn_hi,
                       L.xn_lo, e->st));
  CK(gemm_launch(L.p_lm, nullptr, e->d_status, e->st));
  CK(gemm_fixup_launch(L.p_lm, e->st));
  const int zero = 0;
  CK(cudaMemcpyAsync(e->d_pf_temp, &r.smp.temperature, sizeof(float), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_pf_top_p, &r.smp.top_p, sizeof(float), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_pf_seed, &r.seed, sizeof(uint64_t), cudaMemcpyHostToDevice, e->st));
  CK(cudaMemcpyAsync(e->d_pf_step, &zero, sizeof(int), cudaMemcpyHostToDevice, e->st));
  SampleArgs sa{L.logits, s.vocab, e->d_pf_one, e->d_pf_temp, e->d_pf_top_p, e->d_pf_seed, e->d_pf_step, nullptr,
                e->d_pf_tok};
  CK(launch_sampler(sa, 1, e->st));
  CK(cudaMemcpyAsync(e->pf_logits + (size_t)r.slot * s.vocab, L.logits, (size_t)s.vocab * sizeof(float),
                     cudaMemcpyDeviceToDevice, e->st));
  e->logits_row[(size_t)r.slot] = -1;              // corun_get_logits: the prefill's logits until the slot decodes
  CK(cudaMemcpyAsync(&r.first, e->d_pf_tok, sizeof(int), cudaMemcpyDeviceToHost, e->st));
  CK(cudaStreamSynchronize(e->st));   // the one-row buffers and the sampling staging serve the next request
  return CORUN_OK;
}

// Prefill of one or several requests through the fixed-shape prefill program (chunks of `chunk` rows).  The
// rows of a chunk are dealt in request order; every piece of a request starts on a tile boundary of the
// prefill attention kernel (a tile's rows share one slot), so a chunk may hold pieces of several requests.
// Every kernel of the program treats its rows independently of each other and of where they sit in the
// chunk, and attention reads all keys -- the chunk's own too -- from the cache, so a request's values do not
// depend on how its prompt is cut into pieces nor on what else shares its chunks.
int prefill_run(corun_engine *e, PfReq *reqs, int n_req);

int prefill_many(corun_engine *e, PfReq *reqs, int n_req) {
  RC(sync_stream(e));
  size_t need = 0;
  for (int i = 0; i < n_req; ++i) need += (size_t)(reqs[i].reserve + KV_BLOCK * e->kv_run - 1) / (KV_BLOCK * e->kv_run);   // runs
  if (need > e->free_blocks.size()) return CORUN_ENOSPACE;
  int rc = CORUN_OK;
  for (int i = 0; i < n_req && rc == CORUN_OK; ++i) rc = reserve_blocks(e, reqs[i].slot, reqs[i].reserve);
  if (rc == CORUN_OK) rc = prefill_run(e, reqs, n_req);
  if (rc != CORUN_OK)                               // nothing was admitted: the pages go back to the pool
    for (int i = 0; i < n_req; ++i) {
      std::vector<int> &mine = e->slot_blocks[reqs[i].slot];
      if (e->in_use[reqs[i].slot]) continue;
      for (int b : mine) e->free_blocks.push_back(b);
      mine.clear();
    }
  return rc;
}

int prefill_run(corun_engine *e, PfReq *reqs, int n_req) {
  const corun_shape &s = e->sh;
  Program &P = e->pre;
  const int CH = e->chunk;
  int unit = 128 / (s.n_q_heads / s.n_kv_heads);    // tokens per attention tile
  if (e->mla) unit = 16;                            // no query tiles there: every row is on its own
  if (unit > CH || CH % unit) unit = CH;
  int *tok = e->h_rows, *pos = tok + CH, *act = pos + CH, *slt = act + CH, *blocks = slt + CH;
  std::vector<std::pair<int, int>> fins;           // (request, chunk row of its last prompt token)
  int fill = 0, pad_slot = reqs[0].slot;
  auto run_chunk = [&]() -> int {
    for (int i = fill; i < CH; ++i) { tok[i] = 0; pos[i] = 0; act[i] = 0; slt[i] = pad_slot; }
    CK(cudaMemcpyAsync(P.row_token, tok, CH * sizeof(int), cudaMemcpyHostToDevice, e->st));
    CK(cudaMemcpyAsync(P.row_pos, pos, CH * sizeof(int), cudaMemcpyHostToDevice, e->st));
    CK(cudaMemcpyAsync(P.row_active, act, CH * sizeof(int), cudaMemcpyHostToDevice, e->st));
    CK(cudaMemcpyAsync(P.row_slot, slt, CH * sizeof(int), cudaMemcpyHostToDevice, e->st));
    // the chunk's rows are filled from row 0: the GEMMs leave out the blocks of rows behind the last one in use
    // (blocks of 64 rows up to 128 padded rows, of 128 rows above)
    const int blk = P.BN <= 128 ? 64 : 128;
    blocks[0] = (fill > 0 ? 1 : 0) | (fill > blk ? 2 : 0);
    CK(cudaMemcpyAsync(P.row_blocks, blocks, sizeof(int), cudaMemcpyHostToDevice, e->st));
    RC(run_layers(e, P, nullptr));
    for (auto &f : fins) RC(prefill_finish_row(e, f.second, reqs[f.first]));
    CK(cudaStreamSynchronize(e->st));   // the staging arrays are reused by the next chunk
    fins.clear();
    fill = 0;
    return CORUN_OK;
  };
  for (int r = 0; r < n_req; ++r) {
    const PfReq &q = reqs[r];
    for (int done = 0; done < q.n;) {
      while (fill % unit) { tok[fill] = 0; pos[fill] = 0; act[fill] = 0; slt[fill] = pad_slot; ++fill; }   // rest of the tile before
      if (fill == CH) RC(run_chunk());
      const int take = q.n - done < CH - fill ? q.n - done : CH - fill;
      for (int i = 0; i < take; ++i) {
        tok[fill + i] = q.tokens[done + i];
        pos[fill + i] = done + i;
        act[fill + i] = 1;
        slt[fill + i] = q.slot;
      }
      fill += take;
      done += take;
      pad_slot = q.slot;                            // padding up to the tile's end belongs to this request's tile
      if (done == q.n) fins.emplace_back(r, fill - 1);
      if (fill == CH) RC(run_chunk());
    }
  }
  if (fill > 0 || !fins.empty()) RC(run_chunk());
  CK(cudaMemcpyAsync(e->h_status, e->d_status, sizeof(int), cudaMemcpyDeviceToHost, e->st));
  CK(cudaStreamSynchronize(e->st));
  RC(check_status(e));
  for (int i = 0; i < n_req; ++i) {
    PfReq &q = reqs[i];
    RC(set_slot_state(e, q.slot, 1, q.n, 1, q.first, q.smp.temperature, q.smp.top_p));
    e->in_use[q.slot] = 1;
    e->ctx[q.slot] = q.n;
    e->reserve[q.slot] = q.reserve;
    e->step[q.slot] = 1;
  }
  return CORUN_OK;
}

}  // namespace

extern "C" {

int corun_prefill(corun_engine *e, int32_t slot, const int32_t *tokens, int32_t n, int32_t reserve_len,
                  const corun_sampling *sampling, uint64_t seed, int32_t *out_first_token) {
  if (!e || !tokens || !sampling || n < 1 || reserve_len < n || reserve_len > e->max_ctx) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || e->in_use[slot]) return CORUN_ESLOT;
  for (int i = 0; i < n; ++i)
    if (tokens[i] < 0 || tokens[i] >= e->sh.vocab) return CORUN_EINVAL;
  PfReq r{slot, tokens, n, reserve_len, *sampling, seed, -1};
  RC(prefill_many(e, &r, 1));
  if (out_first_token) *out_first_token = r.first;
  return CORUN_OK;
}

int corun_prefill_batch(corun_engine *e, int32_t n_req, const int32_t *slots, const int32_t *tokens,
                        const int32_t *n_tokens, const int32_t *reserve_lens, const corun_sampling *samplings,
                        const uint64_t *seeds, int32_t *out_first_tokens) {
  if (!e || n_req < 1 || !slots || !tokens || !n_tokens || !reserve_lens || !samplings || !seeds) return CORUN_EINVAL;
  std::vector<PfReq> reqs((size_t)n_req);
  size_t off = 0;
  for (int i = 0; i < n_req; ++i) {
    const int n = n_tokens[i];
    if (n < 1 || reserve_lens[i] < n || reserve_lens[i] > e->max_ctx) return CORUN_EINVAL;
    if (!slot_ok(e, slots[i]) || e->in_use[slots[i]]) return CORUN_ESLOT;
    for (int j = 0; j < i; ++j)
      if (slots[j] == slots[i]) return CORUN_ESLOT;
    for (int t = 0; t < n; ++t)
      if (tokens[off + t] < 0 || tokens[off + t] >= e->sh.vocab) return CORUN_EINVAL;
    reqs[i] = PfReq{slots[i], tokens + off, n, reserve_lens[i], samplings[i], seeds[i], -1};
    off += (size_t)n;
  }
  RC(prefill_many(e, reqs.data(), n_req));
  if (out_first_tokens)
    for (int i = 0; i < n_req; ++i) out_first_tokens[i] = reqs[i].first;
  return CORUN_OK;
}

int corun_decode_enqueue(corun_engine *e, const uint8_t *active, const uint64_t *seeds) {
  if (!e || !active || !seeds) return CORUN_EINVAL;
  for (int s = 0; s < e->B; ++s) {
    if (!active[s]) continue;
    if (!e->in_use[s]) return CORUN_ESLOT;
    if (e->ctx[s] + 1 > e->reserve[s]) return CORUN_ECTX;
  }
  bool same = e->staged_valid;
  for (int s = 0; s < e->B && same; ++s) {
    const uint8_t a = active[s] ? 1 : 0;
    if (e->h_active[s] != a || (a && e->h_seeds[s] != seeds[s])) same = false;
  }
  if (!same) {
    if (e->in_flight) RC(sync_stream(e));   // an earlier replay may still read the staging buffers
    for (int s = 0; s < e->B; ++s) {
      e->h_active[s] = active[s] ? 1 : 0;
      e->h_seeds[s] = active[s] ? seeds[s] : 0;
    }
    e->staged_valid = true;
  }
  if (e->eager) {
    RC(enqueue_decode_body(e, nullptr));
  } else {
    CK(cudaGraphLaunch(e->graph_exec, e->st));
  }
  e->in_flight = true;
  int row = 0;                                      // the step's rows: the slots with a request, ascending (prepare_rows)
  for (int s = 0; s < e->B; ++s)
    if (active[s]) {
      e->ctx[s] += 1;
      e->step[s] += 1;
      e->logits_row[(size_t)s] = row++;
    }
  return CORUN_OK;
}

int corun_decode_wait(corun_engine *e, int32_t *out_tokens) {
  if (!e) return CORUN_EINVAL;
  RC(sync_stream(e));
  if (out_tokens) memcpy(out_tokens, e->h_out_tokens, e->B * sizeof(int));
  return check_status(e);
}

int corun_decode_step(corun_engine *e, const uint8_t *active, const uint64_t *seeds, int32_t *out_tokens) {
  if (!out_tokens) return CORUN_EINVAL;
  RC(corun_decode_enqueue(e, active, seeds));
  return corun_decode_wait(e, out_tokens);
}

int corun_release(corun_engine *e, int32_t slot) {
  if (!e) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  RC(sync_stream(e));
  for (int b : e->slot_blocks[slot]) e->free_blocks.push_back(b);
  e->slot_blocks[slot].clear();
  RC(set_slot_state(e, slot, 0, 0, 0, 0, 0.f, 1.f));
  e->in_use[slot] = 0;
  e->ctx[slot] = 0;
  e->reserve[slot] = 0;
  e->step[slot] = 0;
  return CORUN_OK;
}

int corun_get_logits(corun_engine *e, int32_t slot, float *out) {
  if (!e || !out) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  RC(sync_stream(e));
  // the logits of the slot's newest token: its row of the last decode step it took part in, else its prefill's
  const int row = e->logits_row[(size_t)slot];
  const float *src = row < 0 ? e->pf_logits + (size_t)slot * e->sh.vocab : e->dec.logits + (size_t)row * e->sh.vocab;
  CK(cudaMemcpyAsync(out, src, (size_t)e->sh.vocab * sizeof(float), cudaMemcpyDeviceToHost, e->st));
  CK(cudaStreamSynchronize(e->st));
  return CORUN_OK;
}

int corun_force_token(corun_engine *e, int32_t slot, int32_t token) {
  if (!e || token < 0 || token >= e->sh.vocab) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  RC(sync_stream(e));
  CK(cudaMemcpyAsync(e->d_pending + slot, &token, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaStreamSynchronize(e->st));
  return CORUN_OK;
}

int corun_context_len(corun_engine *e, int32_t slot) {
  if (!e) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  return e->ctx[slot];
}

int64_t corun_free_blocks(corun_engine *e) { return e ? (int64_t)e->free_blocks.size() : (int64_t)CORUN_EINVAL; }

int corun_engine_info(corun_engine *e, int32_t *B, int32_t *max_context, int32_t *kv_block, int64_t *pool_blocks) {
  if (!e) return CORUN_EINVAL;
  if (B) *B = e->B;
  if (max_context) *max_context = e->max_ctx;
  if (kv_block) *kv_block = KV_BLOCK * e->kv_run;   // the unit pages are handed out in (corun_free_blocks counts these)
  if (pool_blocks) *pool_blocks = e->pool_blocks / e->kv_run;
  return CORUN_OK;
}

int corun_prefill_geometry(corun_engine *e, int32_t *chunk_rows, int32_t *tile_rows) {
  if (!e) return CORUN_EINVAL;
  int unit = 128 / (e->sh.n_q_heads / e->sh.n_kv_heads);
  if (e->mla) unit = 16;
  if (unit > e->chunk || e->chunk % unit) unit = e->chunk;
  if (chunk_rows) *chunk_rows = e->chunk;
  if (tile_rows) *tile_rows = unit;
  return CORUN_OK;
}

// MLA engines: k holds the cached rows ([n][rank + rope]), v is not used (may be NULL).
static int latent_io(corun_engine *e, int slot, int layer, int pos0, int n, float *k, int write) {
  const int row = e->md.rank + e->md.rope;
  const size_t elems = (size_t)n * row;
  float *dk = nullptr;
  if (cudaMalloc(&dk, elems * sizeof(float)) != cudaSuccess) return CORUN_ENOMEM;
  const MlaCache cache{e->kv_pool + (size_t)layer * e->layer_stride, e->d_block_table, e->max_blocks, e->B, (long long)e->pool_blocks, e->kv_run};
  cudaError_t ce = cudaSuccess;
  if (write) ce = cudaMemcpyAsync(dk, k, elems * sizeof(float), cudaMemcpyHostToDevice, e->st);
  if (ce == cudaSuccess) ce = launch_mla_copy(cache, row, slot, pos0, n, dk, write, e->st);
  if (ce == cudaSuccess && !write) ce = cudaMemcpyAsync(k, dk, elems * sizeof(float), cudaMemcpyDeviceToHost, e->st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(e->st);
  cudaFree(dk);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return CORUN_OK;
}

static int kv_io(corun_engine *e, int slot, int layer, int pos0, int n, float *k, float *v, int write) {
  if (e && e->mla && !v) v = k;                     // the latent cache has no second array
  if (!e || !k || !v || n < 0 || pos0 < 0 || layer < 0 || layer >= e->sh.n_layers) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  const int limit = write ? e->reserve[slot] : e->ctx[slot];
  if (pos0 + n > limit) return CORUN_EINVAL;
  if (n == 0) return CORUN_OK;
  RC(sync_stream(e));
  if (e->mla) {
    RC(latent_io(e, slot, layer, pos0, n, k, write));
    if (write && pos0 + n > e->ctx[slot]) {
      e->ctx[slot] = pos0 + n;
      const int c = e->ctx[slot];
      CK(cudaMemcpyAsync(e->d_ctx + slot, &c, sizeof(int), cudaMemcpyHostToDevice, e->st));
      CK(cudaStreamSynchronize(e->st));
    }
    return CORUN_OK;
  }
  const size_t elems = (size_t)n * e->sh.n_kv_heads * e->sh.head_dim;
  float *dk = nullptr, *dv = nullptr;
  if (cudaMalloc(&dk, elems * sizeof(float)) != cudaSuccess) return CORUN_ENOMEM;
  if (cudaMalloc(&dv, elems * sizeof(float)) != cudaSuccess) { cudaFree(dk); return CORUN_ENOMEM; }
  int rc = CORUN_OK;
  cudaError_t ce = cudaSuccess;
  // every copy is ordered on the engine's own stream: a host-synchronous cudaMemcpy from pageable
  // memory may return before its DMA has landed, and the engine's stream does not wait for the
  // legacy stream
  if (write) {
    ce = cudaMemcpyAsync(dk, k, elems * sizeof(float), cudaMemcpyHostToDevice, e->st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(dv, v, elems * sizeof(float), cudaMemcpyHostToDevice, e->st);
  }
  if (ce == cudaSuccess) ce = launch_kv_copy(kv_layout(e), layer, slot, pos0, n, dk, dv, write, e->st);
  if (ce == cudaSuccess && !write) {
    ce = cudaMemcpyAsync(k, dk, elems * sizeof(float), cudaMemcpyDeviceToHost, e->st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(v, dv, elems * sizeof(float), cudaMemcpyDeviceToHost, e->st);
  }
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(e->st);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; rc = CORUN_ECUDA; }
  cudaFree(dk);
  cudaFree(dv);
  if (rc == CORUN_OK && write && pos0 + n > e->ctx[slot]) {
    e->ctx[slot] = pos0 + n;
    const int c = e->ctx[slot];
    CK(cudaMemcpyAsync(e->d_ctx + slot, &c, sizeof(int), cudaMemcpyHostToDevice, e->st));
    CK(cudaStreamSynchronize(e->st));
  }
  return rc;
}

int corun_debug_kv_read(corun_engine *e, int32_t slot, int32_t layer, int32_t pos0, int32_t n, float *k, float *v) {
  return kv_io(e, slot, layer, pos0, n, k, v, 0);
}
int corun_debug_kv_write(corun_engine *e, int32_t slot, int32_t layer, int32_t pos0, int32_t n, const float *k,
                         const float *v) {
  return kv_io(e, slot, layer, pos0, n, const_cast<float *>(k), const_cast<float *>(v), 1);
}

int corun_debug_adopt(corun_engine *e, int32_t slot, int32_t n_ctx, int32_t reserve_len, int32_t pending_token,
                      const corun_sampling *sampling, int32_t step) {
  if (!e || !sampling || n_ctx < 0 || reserve_len < n_ctx || reserve_len < 1 || reserve_len > e->max_ctx ||
      pending_token < 0 || pending_token >= e->sh.vocab || step < 0)
    return CORUN_EINVAL;
  if (!slot_ok(e, slot) || e->in_use[slot]) return CORUN_ESLOT;
  RC(sync_stream(e));
  RC(reserve_blocks(e, slot, reserve_len));
  RC(set_slot_state(e, slot, 1, n_ctx, step, pending_token, sampling->temperature, sampling->top_p));
  e->in_use[slot] = 1;
  e->ctx[slot] = n_ctx;
  e->reserve[slot] = reserve_len;
  e->step[slot] = step;
  return CORUN_OK;
}

int corun_debug_kv_fill(corun_engine *e, int32_t slot, int32_t n_ctx, float std, uint64_t seed) {
  if (!e || n_ctx < 0 || !(std >= 0.f)) return CORUN_EINVAL;
  if (!slot_ok(e, slot) || !e->in_use[slot]) return CORUN_ESLOT;
  if (n_ctx > e->reserve[slot]) return CORUN_EINVAL;
  RC(sync_stream(e));
  if (e->mla) {
    for (int l = 0; l < e->sh.n_layers; ++l) {
      const MlaCache cache{e->kv_pool + (size_t)l * e->layer_stride, e->d_block_table, e->max_blocks, e->B, (long long)e->pool_blocks, e->kv_run};
      CK(launch_mla_fill(cache, e->md.rank + e->md.rope, l, slot, n_ctx, std, seed, e->st));
    }
  } else {
    CK(launch_kv_fill(kv_layout(e), e->sh.n_layers, slot, n_ctx, std, seed, e->st));
  }
  CK(cudaMemcpyAsync(e->d_ctx + slot, &n_ctx, sizeof(int), cudaMemcpyHostToDevice, e->st));
  CK(cudaStreamSynchronize(e->st));
  e->ctx[slot] = n_ctx;
  return CORUN_OK;
}

int corun_debug_time_kernel(corun_engine *e, int32_t kind, int32_t reps, float *avg_ms) {
  if (!e || !avg_ms || reps < 1 || kind < 0 || kind > 13) return CORUN_EINVAL;
  if ((kind == 10 || kind == 11) && !e->mla) return CORUN_EINVAL;   // the up-projections of an MLA layer
  if (kind == 12 && !e->moe_E) return CORUN_EINVAL;                  // the router of an expert layer
  if (kind == 13 && !(e->moe_E && e->dec.grouped)) return CORUN_EINVAL;   // grouping + gather of the grouped form
  RC(sync_stream(e));
  Program &P = e->dec;
  const corun_shape &s = e->sh;
  const Rows rows{P.row_token, P.row_pos, P.row_active, P.row_slot, P.R};
  const KvLayout kv = kv_layout(e);
  cudaEvent_t a, b;
  CK(cudaEventCreate(&a));
  CK(cudaEventCreate(&b));
  int rc = CORUN_OK;
  for (int pass = 0; pass < 2 && rc == CORUN_OK; ++pass) {   // pass 0 warms up
    const int n = pass == 0 ? (reps < 3 ? reps : 3) : reps;
    cudaError_t ce = cudaEventRecord(a, e->st);
    for (int i = 0; i < n && ce == cudaSuccess; ++i) {
      int l = i % s.n_layers;         // rotate over the layers so that L2 cannot hold the weights
      // feed-forward kinds of a decoder with dense and expert layers: the expert layers
      if (e->mla && e->moe_E && (kind == 2 || kind == 3 || kind == 6 || kind == 8 || kind == 12 || kind == 13))
        l = e->first_dense + i % (s.n_layers - e->first_dense);
      GemmOut prev = ffn_out(e, P, l);
      const MlaCache mcache{e->mla ? e->kv_pool + (size_t)l * e->layer_stride : nullptr, e->d_block_table, e->max_blocks, e->B,
                            (long long)e->pool_blocks, e->kv_run};
      switch (kind) {
        // launched as in the step's graph: with programmatic stream serialization
        case 0: ce = gemm_launch(P.p_qkv, &e->tm_qkv[l], e->d_status, e->st, nullptr, true); break;
        case 1: ce = gemm_launch(P.p_o, &e->tm_o[l], e->d_status, e->st, nullptr, true); break;
        case 2: if (P.grouped && !dense_layer(e, l)) {   // the groups of the last step's last layer
                  ce = gemm_launch(P.p_gug, P.p_gug.sw_hi ? &e->tm_gu_half[l] : &e->tm_gu[l], e->d_status, e->st, nullptr, true);
                  if (ce == cudaSuccess && !P.p_gug.sw_hi)
                    ce = launch_moe_swiglu_grouped(P.gug_out, P.moe_w, e->moe_E + e->moe_S, e->moe_F, P.grp, P.hg_hi, P.hg_lo, e->st);
                  break;
                }
                ce = gemm_launch(P.p_gu, P.p_gu.sw_hi ? &e->tm_gu_half[l] : &e->tm_gu[l], e->d_status, e->st, nullptr, true); break;
        case 3: if (P.grouped && !dense_layer(e, l)) {   // per-group down GEMM + the sum over a row's experts
                  ce = gemm_launch(P.p_dng, &e->tm_down[l], e->d_status, e->st, nullptr, true);
                  if (ce == cudaSuccess) ce = launch_moe_combine(P.yg_out, P.row_active, P.R, e->moe_E + e->moe_S, s.hidden, P.grp, P.down_out, e->st);
                  break;
                }
                ce = gemm_launch(P.p_down, &e->tm_down[l], e->d_status, e->st, nullptr, true); break;
        case 4: ce = gemm_launch(P.p_lm, nullptr, e->d_status, e->st, nullptr, true);
                if (ce == cudaSuccess) ce = gemm_fixup_launch(P.p_lm, e->st);
                break;
        case 5: if (e->mla) {
                  ce = launch_mla_attention(e->tm_c[l], e->tm_cv[l], P.q_lat, e->md.rank, (long long)P.RPH * e->md.rank, P.q_rope,
                                            e->d_block_table, e->max_blocks, nullptr, &rows, P.R, e->md,
                                            1.0f / sqrtf((float)(e->md.nope + e->md.rope)), e->mla_splits, P.mla_ml, P.mla_po, nullptr,
                                            P.ol_hi, P.ol_lo, P.RPH, e->num_sms, e->d_status, true, e->st, e->kv_run);
                  break;
                }
                ce = cudaMemsetAsync(P.att_pool + l, 0, sizeof(int), e->st);   // the launch does not reset its pool counter
                if (ce == cudaSuccess)
                  ce = launch_attention(e->tm_k4[l], e->tm_k4[l], P.q, rows, s.n_q_heads, kv, l, e->max_splits, P.att_work,
                                        P.att_n_work, e->num_sms, P.part_acc, P.part_ml, P.att_pool + l,
                                        P.ao_hi, P.ao_lo, e->whole_pairs ? 2 : 0, e->d_status, e->st);
                break;
        case 6: ce = launch_resid_norm(P.h, s.hidden, nullptr, rows, &prev, e->attn_norm[l], s.rms_eps, P.xn_hi,
                                       P.xn_lo, e->st); break;
        case 7: if (e->mla) {   // (re-appends the rows' current positions: the same values)
                  ce = launch_mla_post(P.p_qkv.out(), rows, e->d_rope, e->md, e->kv_norm[l], s.rms_eps, mcache, P.RPH, P.qn_hi, P.qn_lo,
                                       P.q_rope, e->d_status, e->st);
                  break;
                }
                ce = launch_qkv_post(P.p_qkv.out(), rows, e->d_rope, s.n_q_heads, kv, l, P.q, e->d_status, e->st); break;
        case 8: if (P.p_gu.sw_hi || P.grouped) break;   // no such kernel: the SwiGLU is in the GEMM's epilogue (grouped form: timed with kind 2)
                ce = e->moe_E ? launch_moe_swiglu(P.p_gu.out(), P.moe_w, P.R, e->moe_F, e->moe_E + e->moe_S, P.ff_hi, P.ff_lo, e->st)
                              : launch_swiglu(P.p_gu.out(), P.R, s.ffn, P.ff_hi, P.ff_lo, e->st);
                break;
        case 9: {
          SampleArgs sa{P.logits, s.vocab, P.do_sample, P.row_temp, P.row_top_p, e->d_seeds, P.row_step, nullptr, P.sampled};
          ce = launch_sampler(sa, P.R, e->st);
          break;
        }
        case 10: ce = gemm_launch(P.p_uk, &e->tm_uk[l], e->d_status, e->st, nullptr, true); break;
        case 11: ce = gemm_launch(P.p_uv, &e->tm_uv[l], e->d_status, e->st, nullptr, true);
                 if (ce == cudaSuccess) ce = launch_mla_ao_split(P.uv_out, P.R, P.RPH, e->md, P.ao_hi, P.ao_lo, e->st);
                 break;
        case 13: ce = launch_moe_group(P.moe_w, P.row_active, P.R, e->moe_E, e->moe_S, e->moe_F, P.grp, e->st);
                 if (ce == cudaSuccess) ce = launch_moe_gather(P.xn_hi, P.xn_lo, s.hidden, P.grp, P.xg_hi, P.xg_lo, e->st);
                 break;
        case 12: ce = launch_moe_router(P.xn_hi, P.xn_lo, s.hidden, e->router[l], P.R, e->moe_E, e->moe_S, e->moe_K, e->moe_renorm,
                                        P.moe_w, nullptr, nullptr, e->st);
                 break;
      }
    }
    if (ce == cudaSuccess) ce = cudaEventRecord(b, e->st);
    if (ce == cudaSuccess) ce = cudaEventSynchronize(b);
    float ms = 0.f;
    if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, a, b);
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; rc = CORUN_ECUDA; }
    *avg_ms = ms / (float)n;
  }
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  return rc;
}

#ifdef CORUN_BUILD_DEBUG   // kernel timelines: not part of the serving build
int corun_debug_gemm_trace(corun_engine *e, int32_t kind, int32_t layer, uint64_t *stamps, int32_t *n_ctas) {
  if (!e || !stamps || !n_ctas || kind < 0 || kind > 4 || layer < 0 || layer >= e->sh.n_layers) return CORUN_EINVAL;
  RC(sync_stream(e));
  Program &P = e->dec;
  const GemmPlan *pl[5] = {&P.p_qkv, &P.p_o, &P.p_gu, &P.p_down, &P.p_lm};
  const CUtensorMap *tm[5] = {&e->tm_qkv[layer], &e->tm_o[layer], P.p_gu.sw_hi ? &e->tm_gu_half[layer] : &e->tm_gu[layer],
                              &e->tm_down[layer], nullptr};
  const GemmPlan &p = *pl[kind];
  unsigned long long *d = nullptr;
  if (cudaMalloc(&d, (size_t)p.grid * 8 * sizeof(unsigned long long)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t ce = cudaMemsetAsync(d, 0, (size_t)p.grid * 8 * sizeof(unsigned long long), e->st);
  for (int i = 0; i < 3 && ce == cudaSuccess; ++i) ce = gemm_launch(p, tm[kind], e->d_status, e->st, d);   // last one counts
  if (ce == cudaSuccess)
    ce = cudaMemcpyAsync(stamps, d, (size_t)p.grid * 8 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, e->st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(e->st);
  cudaFree(d);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  *n_ctas = p.grid;
  return CORUN_OK;
}

int corun_debug_attn_trace(corun_engine *e, int32_t layer, uint64_t *stamps, int32_t *n_ctas) {
  if (!e || !stamps || !n_ctas || layer < 0 || layer >= e->sh.n_layers || e->mla) return CORUN_EINVAL;
  RC(sync_stream(e));
  Program &P = e->dec;
  const corun_shape &s = e->sh;
  const Rows rows{P.row_token, P.row_pos, P.row_active, P.row_slot, P.R};
  const size_t n = (size_t)e->num_sms * 64 * 8;
  unsigned long long *d = nullptr;
  if (cudaMalloc(&d, n * sizeof(unsigned long long)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t ce = cudaMemsetAsync(d, 0, n * sizeof(unsigned long long), e->st);
  for (int i = 0; i < 2 && ce == cudaSuccess; ++i) {
    ce = cudaMemsetAsync(P.att_pool + layer, 0, sizeof(int), e->st);   // the launch does not reset its pool counter
    if (ce == cudaSuccess)
      ce = launch_attention(e->tm_k4[layer], e->tm_k4[layer], P.q, rows, s.n_q_heads, kv_layout(e), layer, e->max_splits,
                            P.att_work, P.att_n_work, e->num_sms, P.part_acc, P.part_ml, P.att_pool + layer,
                            P.ao_hi, P.ao_lo, e->whole_pairs ? 2 : 0, e->d_status, e->st, i == 1 ? d : nullptr);   // only the second launch is recorded
  }
  if (ce == cudaSuccess) ce = cudaMemcpyAsync(stamps, d, n * sizeof(unsigned long long), cudaMemcpyDeviceToHost, e->st);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(e->st);
  cudaFree(d);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  *n_ctas = e->num_sms;
  return CORUN_OK;
}

int corun_debug_step_trace(corun_engine *e, uint64_t *stamps, int64_t n) {
  if (!e || !stamps) return CORUN_EINVAL;
  if (!e->step_trace) return CORUN_EINVAL;    // the engine was not created with CORUN_TRACE_STEP=1
  const int64_t have = (int64_t)4 * e->sh.n_layers * e->num_sms * 8;
  if (n != have) return CORUN_EINVAL;
  RC(sync_stream(e));
  CK(cudaMemcpyAsync(stamps, e->step_trace, (size_t)n * sizeof(uint64_t), cudaMemcpyDeviceToHost, e->st));
  CK(cudaStreamSynchronize(e->st));
  return CORUN_OK;
}

#endif  // CORUN_BUILD_DEBUG

int corun_debug_read(corun_engine *e, int32_t which, float *out, int64_t n) {
  if (!e || !out || n < 0) return CORUN_EINVAL;
  RC(sync_stream(e));
  Program &P = e->dec;
  const corun_shape &s = e->sh;
  const size_t QD = (size_t)s.n_q_heads * s.head_dim;
  const float *src = nullptr;
  size_t have = 0;
  switch (which) {
    case 0: src = P.q; have = (size_t)P.R * QD; break;
    case 1: src = P.part_acc; have = (size_t)P.R * s.n_q_heads * e->max_splits * s.head_dim; break;
    case 2: src = P.part_ml; have = (size_t)P.R * s.n_q_heads * e->max_splits * 2; break;
    case 3: src = P.h; have = (size_t)P.R * s.hidden; break;
    case 4: src = (const float *)P.ao_hi; have = (size_t)P.BN * QD / 2; break;
    case 5: src = (const float *)P.ao_lo; have = (size_t)P.BN * QD / 2; break;
    case 6: src = P.o_out; have = (size_t)P.R * s.hidden; break;
    case 7: src = P.ws; have = gemm_ws_floats(e->num_sms, P.BN); break;
    default: return CORUN_EINVAL;
  }
  if ((size_t)n > have) return CORUN_EINVAL;
  CK(cudaMemcpyAsync(out, src, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, e->st));
  CK(cudaStreamSynchronize(e->st));
  return CORUN_OK;
}

int corun_debug_set_eager(corun_engine *e, int32_t eager) {
  if (!e) return CORUN_EINVAL;
  RC(sync_stream(e));
  e->eager = eager != 0;
  e->stop_after = eager > 1 ? eager - 2 : -1;   // eager = 2 + k: stop the layer stack after k stages
  return CORUN_OK;
}

int corun_decode_launches(corun_engine *e) { return e ? e->decode_launches : CORUN_EINVAL; }

int corun_debug_gemm(const void *W, int32_t N, int32_t K, const float *X, int32_t R, float *out, void *cuda_stream) {
  if (!W || !X || !out || N < 1 || K < 64 || K % 64 || R < 1 || R > 256) return CORUN_EINVAL;
  // 16-byte stores of the output, tensor-map loads of W: misaligned buffers are refused before any launch
  if (((uintptr_t)out & 15u) || ((uintptr_t)W & 15u) || ((uintptr_t)X & 3u)) return CORUN_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int dev = 0, sms = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int BN = pad16(R);
  std::vector<void *> keep;
  bf16 *hi = nullptr, *lo = nullptr;
  float *ws = nullptr;
  int *status = nullptr;
  int rc = CORUN_OK;
  GemmPlan p;
  if ((rc = dmalloc(keep, &hi, (size_t)BN * K)) == 0 && (rc = dmalloc(keep, &lo, (size_t)BN * K)) == 0 &&
      (rc = dmalloc(keep, &ws, gemm_ws_floats(sms, BN))) == 0 && (rc = dmalloc(keep, &status, 1)) == 0 &&
      (rc = gemm_plan_create(&p, W, N, K, hi, lo, R, BN, out, ws, sms)) == 0) {
    cudaError_t ce = cudaDeviceSynchronize();   // allocations were cleared through the legacy stream
    if (ce == cudaSuccess) ce = launch_split(X, R, K, hi, lo, st);
    if (ce == cudaSuccess) ce = gemm_launch(p, nullptr, status, st);
    if (ce == cudaSuccess) ce = gemm_fixup_launch(p, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    int hs = 0;
    if (ce == cudaSuccess) ce = cudaMemcpy(&hs, status, sizeof(int), cudaMemcpyDeviceToHost);
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; rc = CORUN_ECUDA; }
    else if (hs != 0) rc = CORUN_ETIMEOUT;
  }
  gemm_plan_destroy(&p);
  for (void *q : keep) cudaFree(q);
  return rc;
}

int corun_debug_variate(uint64_t seed, uint64_t t, uint32_t *out_u24) {
  if (!out_u24) return CORUN_EINVAL;
  uint32_t *d = nullptr;
  if (cudaMalloc(&d, sizeof(uint32_t)) != cudaSuccess) return CORUN_ENOMEM;
  cudaError_t ce = launch_variate(seed, t, d, nullptr);
  if (ce == cudaSuccess) ce = cudaMemcpy(out_u24, d, sizeof(uint32_t), cudaMemcpyDeviceToHost);
  cudaFree(d);
  if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return CORUN_ECUDA; }
  return CORUN_OK;
}

int corun_debug_sample(const float *logits, int32_t n_rows, int32_t vocab, const corun_sampling *sampling,
                       const uint32_t *u24, int32_t *out_tokens) {
  if (!logits || !sampling || !u24 || !out_tokens || n_rows < 1 || vocab < 1) return CORUN_EINVAL;
  std::vector<void *> keep;
  float *dl = nullptr, *dt = nullptr, *dp = nullptr;
  int *dflag = nullptr, *dstep = nullptr, *dtok = nullptr;
  uint32_t *du = nullptr;
  uint64_t *dseed = nullptr;
  int rc;
  if ((rc = dmalloc(keep, &dl, (size_t)n_rows * vocab, false)) == 0 && (rc = dmalloc(keep, &dt, n_rows)) == 0 &&
      (rc = dmalloc(keep, &dp, n_rows)) == 0 && (rc = dmalloc(keep, &dflag, n_rows)) == 0 &&
      (rc = dmalloc(keep, &dstep, n_rows)) == 0 && (rc = dmalloc(keep, &dtok, n_rows)) == 0 &&
      (rc = dmalloc(keep, &du, n_rows)) == 0 && (rc = dmalloc(keep, &dseed, n_rows)) == 0) {
    std::vector<float> t(n_rows, sampling->temperature), p(n_rows, sampling->top_p);
    std::vector<int> ones(n_rows, 1);
    cudaError_t ce = cudaMemcpy(dl, logits, (size_t)n_rows * vocab * sizeof(float), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemcpy(dt, t.data(), n_rows * sizeof(float), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemcpy(dp, p.data(), n_rows * sizeof(float), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemcpy(dflag, ones.data(), n_rows * sizeof(int), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemcpy(du, u24, n_rows * sizeof(uint32_t), cudaMemcpyHostToDevice);
    SampleArgs sa{dl, vocab, dflag, dt, dp, dseed, dstep, du, dtok};
    if (ce == cudaSuccess) ce = launch_sampler(sa, n_rows, nullptr);
    if (ce == cudaSuccess) ce = cudaMemcpy(out_tokens, dtok, n_rows * sizeof(int), cudaMemcpyDeviceToHost);
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; rc = CORUN_ECUDA; }
  }
  for (void *q : keep) cudaFree(q);
  return rc;
}

}  // extern "C"
