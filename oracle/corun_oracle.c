/*
 * CPU oracle for the CoRun hot path: the per-request decoder forward pass
 * (isolated prefill and one decode token), the request-bound random variate
 * R(seed, t) and the deterministic sampling function S.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is deliberately plain and slow, shares no
 * code with the CUDA path, and must never be reached from the product path.
 *
 * What it computes (paper: Background "LLM Inference and Continuous Batching",
 * Design "Determinism Contract", "Isolated Prefill", "Fixed-Shape Batched
 * Decode", "Shape-Aligned Sampling", "Determinism Argument"):
 *   a request's logits are those of the decoder forward pass of that request
 *   alone (request isolation), so the oracle is the textbook definition of a
 *   pre-norm GQA decoder with RoPE and a SwiGLU FFN, evaluated per request with
 *   no batching, paging, graph or split logic.
 *
 * Precision: weights are bf16 bit patterns widened exactly; activations and
 * the KV cache are stored in fp32; every reduction (dot product, mean of
 * squares, softmax sum, weighted value sum) accumulates in fp64 in plain index
 * order.  The only loop liberty taken: a matrix product evaluates several
 * independent rows of activations per weight row at once (each output element
 * is still one index-ordered fp64 sum), and OpenMP distributes independent
 * output elements over cores.  No reduction is blocked, split or reordered.
 *
 * Pins (tests/test_oracle_*.py): brute-force attention and closed forms, RoPE
 * norm and relative-position invariants, RMSNorm/SiLU closed forms, fp64 triple
 * loop GEMM, prefill/decode cache consistency, row independence, degenerate
 * network closed form, a library decoder on the tiny shape, Philox known
 * answers, sampler limits and frequencies.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  float rms_eps, rope_theta;
} orc_shape;

typedef struct {
  const uint16_t *embed;      /* [vocab, hidden]                      */
  const uint16_t *lm_head;    /* [vocab, hidden]                      */
  const uint16_t *final_norm; /* [hidden]                             */
  const uint16_t *const *attn_norm; /* L x [hidden]                   */
  const uint16_t *const *wqkv;      /* L x [(nq+2nkv)*hd, hidden]     */
  const uint16_t *const *wo;        /* L x [hidden, nq*hd]            */
  const uint16_t *const *mlp_norm;  /* L x [hidden]                   */
  const uint16_t *const *wgate_up;  /* L x [2*ffn, hidden]            */
  const uint16_t *const *wdown;     /* L x [hidden, ffn]              */
} orc_weights;

static inline double bf16_to_f64(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* ---- elementary operators (exported so the pins can reach each one) ---- */

/* out[r,n] = sum_k W[n,k] * X[r,k], k ascending, fp64 accumulator. */
void orc_matmul_bf16(const uint16_t *W, int64_t N, int64_t K, const float *X, int64_t R, float *out) {
  enum { RB = 8 };
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    const uint16_t *w = W + n * K;
    for (int64_t r0 = 0; r0 < R; r0 += RB) {
      int64_t rb = R - r0 < RB ? R - r0 : RB;
      double acc[RB];
      for (int j = 0; j < RB; ++j) acc[j] = 0.0;
      if (rb == RB) {
        for (int64_t k = 0; k < K; ++k) {
          double wk = bf16_to_f64(w[k]);
          for (int j = 0; j < RB; ++j) acc[j] += wk * (double)X[(r0 + j) * K + k];
        }
      } else {
        for (int64_t k = 0; k < K; ++k) {
          double wk = bf16_to_f64(w[k]);
          for (int64_t j = 0; j < rb; ++j) acc[j] += wk * (double)X[(r0 + j) * K + k];
        }
      }
      for (int64_t j = 0; j < rb; ++j) out[(r0 + j) * N + n] = (float)acc[j];
    }
  }
}

/* out_i = x_i * g_i / sqrt(mean_j x_j^2 + eps) */
void orc_rmsnorm(const float *x, const uint16_t *g, int64_t H, float eps, float *out) {
  double ss = 0.0;
  for (int64_t i = 0; i < H; ++i) ss += (double)x[i] * (double)x[i];
  double inv = 1.0 / sqrt(ss / (double)H + (double)eps);
  for (int64_t i = 0; i < H; ++i) out[i] = (float)((double)x[i] * inv * bf16_to_f64(g[i]));
}

/* Half-split rotary embedding of one head vector at position pos:
 * pair (i, i+hd/2) is rotated by the angle pos * theta^(-2i/hd). */
void orc_rope(float *v, int32_t head_dim, int64_t pos, float theta) {
  int32_t half = head_dim / 2;
  for (int32_t i = 0; i < half; ++i) {
    double freq = pow((double)theta, -2.0 * (double)i / (double)head_dim);
    double ang = (double)pos * freq;
    double c = cos(ang), s = sin(ang);
    double a = v[i], b = v[i + half];
    v[i] = (float)(a * c - b * s);
    v[i + half] = (float)(a * s + b * c);
  }
}

double orc_silu(double z) { return z / (1.0 + exp(-z)); }

/* Causal softmax attention of one query token at position p over cached
 * positions 0..p (its own key included).  q: [nq, hd]; K, V: rows of
 * nkv*hd floats with stride `stride` floats between positions. */
void orc_attention(const float *q, const float *K, const float *V, int64_t stride, int64_t p,
                   int32_t nq, int32_t nkv, int32_t hd, float *out) {
  int32_t group = nq / nkv;
  double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for schedule(static)
  for (int32_t j = 0; j < nq; ++j) {
    int32_t g = j / group;
    double *s = (double *)malloc(sizeof(double) * (size_t)(p + 1));
    double m = -INFINITY;
    for (int64_t t = 0; t <= p; ++t) {
      const float *k = K + t * stride + (int64_t)g * hd;
      double d = 0.0;
      for (int32_t i = 0; i < hd; ++i) d += (double)q[j * hd + i] * (double)k[i];
      s[t] = d * scale;
      if (s[t] > m) m = s[t];
    }
    double z = 0.0;
    for (int64_t t = 0; t <= p; ++t) {
      s[t] = exp(s[t] - m);
      z += s[t];
    }
    for (int32_t i = 0; i < hd; ++i) {
      double o = 0.0;
      for (int64_t t = 0; t <= p; ++t) o += s[t] * (double)V[t * stride + (int64_t)g * hd + i];
      out[j * hd + i] = (float)(o / z);
    }
    free(s);
  }
}

/* ---- the forward pass ---- */

/*
 * Optional Mixture-of-Experts feed-forward layers (the paper evaluates MoE
 * models -- Evaluation, "Setup" -- without giving formulas; this is the
 * standard block, restated from oracle/moe_oracle.py's definition):
 *   p = softmax(Wr x) over all E experts; S = top_k by p, ties to the lower
 *   id; weights p_e as they are or, with renormalize, divided by their sum
 *   taken in descending-probability order; shared experts always on, weight 1;
 *   y = sum over S in ascending expert id of w_e FFN_e(x), shared experts last;
 *   FFN_e(x) = Wd_e (silu(Wg_e x) * (Wu_e x)).
 * Weight layout per layer: router [E, H]; gate_up [(E + S) * 2F, H], block e =
 * expert e (gate rows, then up rows; shared experts behind the routed ones);
 * down [H, (E + S) * F], columns e*F.. of expert e.
 */
typedef struct {
  int32_t n_experts, top_k, expert_ffn, n_shared, renormalize;
  const uint16_t *const *router;   /* L x [E, H]             */
  const uint16_t *const *gate_up;  /* L x [(E+S)*2F, H]      */
  const uint16_t *const *down;     /* L x [H, (E+S)*F]       */
} orc_moe;

/* One row through one MoE layer: x [H] -> y [H]; ids / probs [top_k] (may be NULL) receive the routing.
 * Everything accumulates in fp64; the hidden activations of an expert are kept in fp64 too. */
void orc_moe_ffn(const orc_moe *m, int64_t layer, int64_t H, const float *x, float *y, int32_t *ids, double *probs) {
  const int64_t E = m->n_experts, F = m->expert_ffn, S = m->n_shared, Kt = m->top_k, NB = E + S;
  const uint16_t *Wr = m->router[layer], *Wgu = m->gate_up[layer], *Wd = m->down[layer];
  double *p = (double *)malloc(sizeof(double) * E);
  double *wt = (double *)calloc((size_t)NB, sizeof(double));
  double *hid = (double *)malloc(sizeof(double) * F);
  double *acc = (double *)calloc((size_t)H, sizeof(double));
  char *taken = (char *)calloc((size_t)E, 1);
  double mx = -INFINITY, sum = 0.0;
  for (int64_t e = 0; e < E; ++e) {
    double d = 0.0;
    for (int64_t i = 0; i < H; ++i) d += bf16_to_f64(Wr[e * H + i]) * (double)x[i];
    p[e] = d;
    if (d > mx) mx = d;
  }
  for (int64_t e = 0; e < E; ++e) { p[e] = exp(p[e] - mx); sum += p[e]; }
  for (int64_t e = 0; e < E; ++e) p[e] /= sum;
  double picked = 0.0;
  int32_t chosen[64];
  for (int64_t k = 0; k < Kt && k < 64; ++k) {
    int64_t best = -1;
    for (int64_t e = 0; e < E; ++e)
      if (!taken[e] && (best < 0 || p[e] > p[best])) best = e;   /* strict: the lower id keeps a tie */
    taken[best] = 1;
    chosen[k] = (int32_t)best;
    picked += p[best];
  }
  for (int64_t k = 0; k < Kt && k < 64; ++k) {
    const double w = m->renormalize ? p[chosen[k]] / picked : p[chosen[k]];
    wt[chosen[k]] = w;
    if (ids) ids[k] = chosen[k];
    if (probs) probs[k] = w;
  }
  for (int64_t s = 0; s < S; ++s) wt[E + s] = 1.0;
  for (int64_t e = 0; e < NB; ++e) {              /* ascending expert id, shared experts last */
    if (e < E && !taken[e]) continue;
    for (int64_t f = 0; f < F; ++f) {
      double g = 0.0, u = 0.0;
      const uint16_t *wg = Wgu + (e * 2 * F + f) * H, *wu = Wgu + (e * 2 * F + F + f) * H;
      for (int64_t i = 0; i < H; ++i) { g += bf16_to_f64(wg[i]) * (double)x[i]; u += bf16_to_f64(wu[i]) * (double)x[i]; }
      hid[f] = orc_silu(g) * u;
    }
    for (int64_t i = 0; i < H; ++i) {
      double d = 0.0;
      const uint16_t *wd = Wd + i * NB * F + e * F;
      for (int64_t f = 0; f < F; ++f) d += bf16_to_f64(wd[f]) * hid[f];
      acc[i] += wt[e] * d;
    }
  }
  for (int64_t i = 0; i < H; ++i) y[i] = (float)acc[i];
  free(p); free(wt); free(hid); free(acc); free(taken);
}

/*
 * Runs tokens[0..T) of ONE request at positions pos0..pos0+T-1 through the
 * decoder.  Kc/Vc: the request's cache, [L][max_T][nkv*hd] fp32; positions
 * below pos0 must already be filled, positions pos0.. are written.
 * logits: [T, vocab] if all_logits, else [vocab] for the last token; may be
 * NULL to skip the LM head.  Returns 0, or -1 on a bad argument.
 * Prefill is T = prompt length at pos0 = 0; a decode step is T = 1.
 */
int orc_forward_ex(const orc_shape *sh, const orc_weights *w, const orc_moe *moe, const int32_t *tokens, int64_t T,
                   int64_t pos0, float *Kc, float *Vc, int64_t max_T, float *logits, int all_logits) {
  const int64_t H = sh->hidden, nq = sh->n_q_heads, nkv = sh->n_kv_heads, hd = sh->head_dim;
  const int64_t F = sh->ffn, Vn = sh->vocab, L = sh->n_layers;
  const int64_t QD = nq * hd, KD = nkv * hd, QKV = QD + 2 * KD;
  if (T <= 0 || pos0 < 0 || pos0 + T > max_T || nq % nkv || hd % 2) return -1;
  for (int64_t t = 0; t < T; ++t)
    if (tokens[t] < 0 || tokens[t] >= Vn) return -1;

  float *h = (float *)malloc(sizeof(float) * T * H);
  float *a = (float *)malloc(sizeof(float) * T * (H > F ? H : F));
  float *qkv = (float *)malloc(sizeof(float) * T * QKV);
  float *o = (float *)malloc(sizeof(float) * T * QD);
  float *y = (float *)malloc(sizeof(float) * T * H);
  float *gu = (float *)malloc(sizeof(float) * T * 2 * F);

  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < H; ++i) h[t * H + i] = (float)bf16_to_f64(w->embed[(int64_t)tokens[t] * H + i]);

  for (int64_t l = 0; l < L; ++l) {
    float *Kl = Kc + l * max_T * KD, *Vl = Vc + l * max_T * KD;
    for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->attn_norm[l], H, sh->rms_eps, a + t * H);
    orc_matmul_bf16(w->wqkv[l], QKV, H, a, T, qkv);
    for (int64_t t = 0; t < T; ++t) {
      float *row = qkv + t * QKV;
      int64_t p = pos0 + t;
      for (int64_t j = 0; j < nq; ++j) orc_rope(row + j * hd, (int32_t)hd, p, sh->rope_theta);
      for (int64_t g = 0; g < nkv; ++g) orc_rope(row + QD + g * hd, (int32_t)hd, p, sh->rope_theta);
      memcpy(Kl + p * KD, row + QD, sizeof(float) * KD);
      memcpy(Vl + p * KD, row + QD + KD, sizeof(float) * KD);
    }
    for (int64_t t = 0; t < T; ++t)
      orc_attention(qkv + t * QKV, Kl, Vl, KD, pos0 + t, (int32_t)nq, (int32_t)nkv, (int32_t)hd, o + t * QD);
    orc_matmul_bf16(w->wo[l], H, QD, o, T, y);
    for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
    for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->mlp_norm[l], H, sh->rms_eps, a + t * H);
    if (moe) {                                      /* Mixture-of-Experts feed-forward layer */
#pragma omp parallel for schedule(dynamic)
      for (int64_t t = 0; t < T; ++t) orc_moe_ffn(moe, l, H, a + t * H, y + t * H, NULL, NULL);
      for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
      continue;
    }
    orc_matmul_bf16(w->wgate_up[l], 2 * F, H, a, T, gu);
    for (int64_t t = 0; t < T; ++t)
      for (int64_t i = 0; i < F; ++i) {
        double g = gu[t * 2 * F + i], u = gu[t * 2 * F + F + i];
        a[t * F + i] = (float)(orc_silu(g) * u);
      }
    orc_matmul_bf16(w->wdown[l], H, F, a, T, y);
    for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
  }

  if (logits) {
    if (all_logits) {
      for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->final_norm, H, sh->rms_eps, a + t * H);
      orc_matmul_bf16(w->lm_head, Vn, H, a, T, logits);
    } else {
      orc_rmsnorm(h + (T - 1) * H, w->final_norm, H, sh->rms_eps, a);
      orc_matmul_bf16(w->lm_head, Vn, H, a, 1, logits);
    }
  }
  free(h); free(a); free(qkv); free(o); free(y); free(gu);
  return 0;
}

/* ---- multi-head latent attention (MLA) decoder ----
 *
 * The paper evaluates one model with MLA and Mixture-of-Experts layers (Evaluation, "Setup") without giving
 * the layer's formulas; this is the published definition of that layer, in the form that caches one latent
 * vector per token (the same definition oracle/mla_oracle.py states for a single query):
 *   a = RMSNorm(h);  [q | kv_a] = W_qkv a,  q: nh heads of (nope + rope) dims,  kv_a: rank + rope dims
 *   c_t = RMSNorm(kv_a[:rank]) * g_kv            the cached latent of the token
 *   r_t = RoPE(kv_a[rank:], t)                   the cached rotary key, shared by all heads
 *   per head h, with W_kv_b's block h = [W_uk (nope rows) ; W_uv (v rows)], both [.., rank]:
 *     k_nope[t] = W_uk c_t,  v[t] = W_uv c_t
 *     s_t = (q_nope . k_nope[t] + RoPE(q_rope, p) . r_t) / sqrt(nope + rope),  t = 0..p
 *     o_h = sum_t softmax(s)_t v[t]
 *   y = W_o [o_0 | o_1 | ...]
 * RoPE is the half-split rotation of orc_rope on the rope dims.  Layers below first_dense have the dense SwiGLU
 * feed-forward of orc_forward_ex (width sh->ffn), the others the Mixture-of-Experts block (moe may be NULL: all
 * layers dense).  sh->n_q_heads = nh; sh->n_kv_heads and sh->head_dim are not used.
 */
typedef struct {
  int32_t kv_lora_rank, qk_nope, qk_rope, v_head, first_dense;
  const uint16_t *const *kv_norm; /* L x [rank]                      */
  const uint16_t *const *wkv_b;   /* L x [nh * (nope + v), rank]     */
} orc_mla;

/* One query token at position p over cached rows 0..p.  q: [nh][nope + rope] (rope part already rotated);
 * Cc: cache rows of rank + rope floats, `stride` floats apart; out: [nh][v]. */
void orc_mla_attention(const float *q, const float *Cc, int64_t stride, int64_t p, int32_t nh, int32_t rank,
                       int32_t nope, int32_t rope, int32_t vh, const uint16_t *wkv_b, float *out) {
  const double scale = 1.0 / sqrt((double)(nope + rope));
#pragma omp parallel for schedule(static)
  for (int32_t h = 0; h < nh; ++h) {
    const uint16_t *Wuk = wkv_b + (int64_t)h * (nope + vh) * rank, *Wuv = Wuk + (int64_t)nope * rank;
    const float *qh = q + (int64_t)h * (nope + rope);
    double *s = (double *)malloc(sizeof(double) * (size_t)(p + 1));
    double *kn = (double *)malloc(sizeof(double) * (size_t)nope);
    double m = -INFINITY;
    for (int64_t t = 0; t <= p; ++t) {
      const float *c = Cc + t * stride;
      double d = 0.0;
      for (int32_t i = 0; i < nope; ++i) {            /* k_nope[t] = W_uk c_t, then its product with q_nope */
        double k = 0.0;
        for (int32_t j = 0; j < rank; ++j) k += bf16_to_f64(Wuk[(int64_t)i * rank + j]) * (double)c[j];
        kn[i] = k;
      }
      for (int32_t i = 0; i < nope; ++i) d += (double)qh[i] * kn[i];
      for (int32_t i = 0; i < rope; ++i) d += (double)qh[nope + i] * (double)c[rank + i];
      s[t] = d * scale;
      if (s[t] > m) m = s[t];
    }
    double z = 0.0;
    for (int64_t t = 0; t <= p; ++t) { s[t] = exp(s[t] - m); z += s[t]; }
    for (int32_t i = 0; i < vh; ++i) {
      double o = 0.0;
      for (int64_t t = 0; t <= p; ++t) {              /* v[t] = W_uv c_t, weighted */
        const float *c = Cc + t * stride;
        double v = 0.0;
        for (int32_t j = 0; j < rank; ++j) v += bf16_to_f64(Wuv[(int64_t)i * rank + j]) * (double)c[j];
        o += s[t] * v;
      }
      out[(int64_t)h * vh + i] = (float)(o / z);
    }
    free(s); free(kn);
  }
}

/* As orc_forward_ex for the MLA decoder.  Cc: the request's cache, [L][max_T][rank + rope] fp32. */
int orc_forward_mla(const orc_shape *sh, const orc_weights *w, const orc_mla *ml, const orc_moe *moe,
                    const int32_t *tokens, int64_t T, int64_t pos0, float *Cc, int64_t max_T, float *logits,
                    int all_logits) {
  const int64_t H = sh->hidden, nh = sh->n_q_heads, F = sh->ffn, Vn = sh->vocab, L = sh->n_layers;
  const int64_t rank = ml->kv_lora_rank, nope = ml->qk_nope, rope = ml->qk_rope, vh = ml->v_head;
  const int64_t QD = nh * (nope + rope), CD = rank + rope, QKV = QD + CD, OD = nh * vh;
  if (T <= 0 || pos0 < 0 || pos0 + T > max_T || rope % 2 || ml->first_dense < 0 || (!moe && ml->first_dense < L)) return -1;
  for (int64_t t = 0; t < T; ++t)
    if (tokens[t] < 0 || tokens[t] >= Vn) return -1;
  int64_t wide = H > F ? H : F;
  float *h = (float *)malloc(sizeof(float) * T * H);
  float *a = (float *)malloc(sizeof(float) * T * wide);
  float *qkv = (float *)malloc(sizeof(float) * T * QKV);
  float *o = (float *)malloc(sizeof(float) * T * OD);
  float *y = (float *)malloc(sizeof(float) * T * H);
  float *gu = (float *)malloc(sizeof(float) * T * 2 * F);
  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < H; ++i) h[t * H + i] = (float)bf16_to_f64(w->embed[(int64_t)tokens[t] * H + i]);
  for (int64_t l = 0; l < L; ++l) {
    float *Cl = Cc + l * max_T * CD;
    for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->attn_norm[l], H, sh->rms_eps, a + t * H);
    orc_matmul_bf16(w->wqkv[l], QKV, H, a, T, qkv);
    for (int64_t t = 0; t < T; ++t) {
      float *row = qkv + t * QKV;
      const int64_t p = pos0 + t;
      for (int64_t j = 0; j < nh; ++j) orc_rope(row + j * (nope + rope) + nope, (int32_t)rope, p, sh->rope_theta);
      orc_rmsnorm(row + QD, ml->kv_norm[l], rank, sh->rms_eps, Cl + p * CD);
      orc_rope(row + QD + rank, (int32_t)rope, p, sh->rope_theta);
      memcpy(Cl + p * CD + rank, row + QD + rank, sizeof(float) * rope);
    }
    for (int64_t t = 0; t < T; ++t)
      orc_mla_attention(qkv + t * QKV, Cl, CD, pos0 + t, (int32_t)nh, (int32_t)rank, (int32_t)nope, (int32_t)rope,
                        (int32_t)vh, ml->wkv_b[l], o + t * OD);
    orc_matmul_bf16(w->wo[l], H, OD, o, T, y);
    for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
    for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->mlp_norm[l], H, sh->rms_eps, a + t * H);
    if (l >= ml->first_dense) {                     /* Mixture-of-Experts feed-forward layer */
#pragma omp parallel for schedule(dynamic)
      for (int64_t t = 0; t < T; ++t) orc_moe_ffn(moe, l, H, a + t * H, y + t * H, NULL, NULL);
      for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
      continue;
    }
    orc_matmul_bf16(w->wgate_up[l], 2 * F, H, a, T, gu);
    for (int64_t t = 0; t < T; ++t)
      for (int64_t i = 0; i < F; ++i) {
        double g = gu[t * 2 * F + i], u = gu[t * 2 * F + F + i];
        a[t * F + i] = (float)(orc_silu(g) * u);
      }
    orc_matmul_bf16(w->wdown[l], H, F, a, T, y);
    for (int64_t i = 0; i < T * H; ++i) h[i] = h[i] + y[i];
  }
  if (logits) {
    if (all_logits) {
      for (int64_t t = 0; t < T; ++t) orc_rmsnorm(h + t * H, w->final_norm, H, sh->rms_eps, a + t * H);
      orc_matmul_bf16(w->lm_head, Vn, H, a, T, logits);
    } else {
      orc_rmsnorm(h + (T - 1) * H, w->final_norm, H, sh->rms_eps, a);
      orc_matmul_bf16(w->lm_head, Vn, H, a, 1, logits);
    }
  }
  free(h); free(a); free(qkv); free(o); free(y); free(gu);
  return 0;
}

int orc_forward(const orc_shape *sh, const orc_weights *w, const int32_t *tokens, int64_t T, int64_t pos0,
                float *Kc, float *Vc, int64_t max_T, float *logits, int all_logits) {
  return orc_forward_ex(sh, w, NULL, tokens, T, pos0, Kc, Vc, max_T, logits, all_logits);
}

/* ---- request-bound random variate R(seed, t) ---- */

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random
 * numbers: as easy as 1, 2, 3", SC'11): multipliers 0xD2511F53 / 0xCD9E8D57,
 * key schedule increments 0x9E3779B9 / 0xBB67AE85. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* R(seed, t): the top 24 bits of the first Philox word with key = seed and
 * counter = (t, 0, 0, 0); the variate is u24 / 2^24 in [0, 1).  Stateless, so
 * padding cannot consume it and moving slots cannot shift it. */
uint32_t orc_variate_u24(uint64_t seed, uint64_t t) {
  uint32_t ctr[4] = {(uint32_t)t, (uint32_t)(t >> 32), 0u, 0u};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  orc_philox4x32_10(ctr, key, out);
  return out[0] >> 8;
}

/* ---- sampling function S ---- */

typedef struct {
  int64_t idx;
  float logit;
} orc_item;

static int orc_item_desc(const void *pa, const void *pb) {
  const orc_item *a = (const orc_item *)pa, *b = (const orc_item *)pb;
  if (a->logit > b->logit) return -1;
  if (a->logit < b->logit) return 1;
  return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

/*
 * exp2 as S defines it: fp32, round-to-nearest-even split x = n + f with
 * |f| <= 1/2, then the degree-7 Taylor polynomial of 2^f (coefficients
 * ln(2)^k / k! rounded to fp32) in Horner form with separately rounded
 * multiplies and adds (no fused multiply-add), then the exact scaling by 2^n.
 * Spelling the arithmetic out makes the integer weights below reproducible bit
 * for bit on any IEEE-754 machine, so that the sampling decision (an integer) is
 * taken in one stated precision by every implementation.  Relative error < 1e-7.
 */
static float orc_pexp2_mantissa(float x, int *n_out) {
  static const float c[8] = {1.0f, 0x1.62e430p-1f, 0x1.ebfbe0p-3f, 0x1.c6b08ep-5f, 0x1.3b2ab6p-7f,
                             0x1.5d87fep-10f, 0x1.430912p-13f, 0x1.ffcbfcp-17f};
  float n = rintf(x);
  float f = x - n;
  float p = c[7];
  for (int k = 6; k >= 0; --k) {
    float t = p * f;
    p = t + c[k];
  }
  *n_out = (int)n;
  return p;
}

/* weight = floor(2^40 * 2^x) for x <= 0, x in fp32 */
uint64_t orc_weight(float logit, float max_logit, float inv_t_log2e) {
  float d = logit - max_logit;
  float x = d * inv_t_log2e;
  if (!(x > -64.0f)) return 0;
  int n;
  float p = orc_pexp2_mantissa(x, &n);
  if (n < -41) return 0;
  return (uint64_t)ldexpf(p, n + 40);      /* exact scaling, then truncation */
}

/*
 * S(logits, u24).  temperature == 0: argmax, lowest id on ties.  Otherwise:
 *   weight_i = floor(2^40 * exp2(fl32(fl32(logit_i - max) * fl32(log2(e) / temperature))))
 *              with exp2 as defined above (integer; equals floor(2^40 * exp((logit_i - max)/T))
 *              up to a relative 2e-7)
 *   total    = sum_i weight_i ;  cut = floor(top_p * total)   (fp64 product)
 *   nucleus  = tokens in descending logit order (ties: lower id first) up to
 *              and including the first whose running weight sum >= cut
 *   Z = nucleus weight ;  r = floor(u24 * Z / 2^24)
 *   token    = first nucleus member, in ascending id order, whose running
 *              weight sum exceeds r.
 * The weights are integers in a stated fp32 arithmetic, so every decision is
 * exact and any implementation must return the same token.  `margin`
 * (optional) receives how close, relative to `total`, the decision came to
 * flipping (min of: distance of r to the nearest running-sum boundary,
 * distance of the cut to the running sums adjacent to the nucleus edge).
 */
int32_t orc_sample(const float *logits, int64_t V, float temperature, float top_p, uint32_t u24, double *margin) {
  int64_t best = 0;
  for (int64_t i = 1; i < V; ++i)
    if (logits[i] > logits[best]) best = i;
  if (margin) *margin = 1.0;
  if (temperature <= 0.0f) return (int32_t)best;

  const float mx = logits[best];
  const float inv_t_log2e = 0x1.715476p+0f / temperature;
  uint64_t *wgt = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)V);
  orc_item *it = (orc_item *)malloc(sizeof(orc_item) * (size_t)V);
  uint64_t total = 0;
  for (int64_t i = 0; i < V; ++i) {
    wgt[i] = orc_weight(logits[i], mx, inv_t_log2e);
    total += wgt[i];
    it[i].idx = i;
    it[i].logit = logits[i];
  }
  qsort(it, (size_t)V, sizeof(orc_item), orc_item_desc);
  uint64_t cut = (uint64_t)floor((double)top_p * (double)total);
  if (cut > total) cut = total;
  char *in = (char *)calloc((size_t)V, 1);
  uint64_t run = 0, Z = 0;
  double mg = 1.0;
  for (int64_t r = 0; r < V; ++r) {
    uint64_t before = run;
    run += wgt[it[r].idx];
    in[it[r].idx] = 1;
    if (run >= cut) {
      Z = run;
      double d1 = (double)(run - cut) / (double)total;          /* cut just reached        */
      double d0 = (double)(cut - before) / (double)total;       /* cut not reached before  */
      mg = d1 < d0 ? d1 : d0;
      if (cut >= total) mg = 1.0;  /* everything is kept: no edge to flip */
      break;
    }
  }
  unsigned __int128 prod = (unsigned __int128)u24 * (unsigned __int128)Z;
  uint64_t rdraw = (uint64_t)(prod >> 24);
  int32_t tok = -1;
  run = 0;
  for (int64_t i = 0; i < V; ++i) {
    if (!in[i]) continue;
    uint64_t before = run;
    run += wgt[i];
    if (run > rdraw) {
      tok = (int32_t)i;
      double d0 = (double)(rdraw - before) / (double)total;
      double d1 = (double)(run - rdraw) / (double)total;
      if (d0 < mg) mg = d0;
      if (d1 < mg) mg = d1;
      break;
    }
  }
  if (margin) *margin = mg;
  free(wgt); free(it); free(in);
  return tok;
}

/*
 * The plain definition of S, kept beside the integer specification above as its pin: everything in fp64 with
 * the C library's exp, no integers.
 *   p_i     = exp((logit_i - max) / temperature)
 *   nucleus = tokens in descending logit order (ties: lower id first) up to and including the first whose
 *             running sum of p reaches top_p * sum_i p_i
 *   token   = first nucleus member, in ascending id order, whose running sum of p exceeds u * Z,
 *             u = u24 / 2^24, Z = nucleus mass.
 * `margin` receives how close, relative to sum_i p_i, any of these comparisons came to going the other way.
 * The integer specification must give the same token whenever the margin exceeds the accuracy of its weights
 * (2e-7 relative per weight, hence per running sum); tests/test_oracle_sampler.py checks exactly that.
 * orc_sample_plain_many / orc_sample_many evaluate n variates against one row (the row is sorted once).
 */
typedef struct {
  int64_t V, n_in;
  double total, Z, edge_margin;
  double *p;       /* per token */
  char *in;        /* nucleus membership */
} orc_plain_row;

static void orc_plain_prepare(orc_plain_row *R, const float *logits, int64_t V, float temperature, float top_p) {
  int64_t best = 0;
  for (int64_t i = 1; i < V; ++i)
    if (logits[i] > logits[best]) best = i;
  R->V = V;
  R->p = (double *)malloc(sizeof(double) * (size_t)V);
  R->in = (char *)calloc((size_t)V, 1);
  orc_item *it = (orc_item *)malloc(sizeof(orc_item) * (size_t)V);
  double total = 0.0;
  for (int64_t i = 0; i < V; ++i) {
    R->p[i] = exp(((double)logits[i] - (double)logits[best]) / (double)temperature);
    it[i].idx = i;
    it[i].logit = logits[i];
  }
  qsort(it, (size_t)V, sizeof(orc_item), orc_item_desc);
  for (int64_t r = 0; r < V; ++r) total += R->p[it[r].idx];   /* summed in the order the nucleus is built in */
  const double cut = (double)top_p * total;
  double run = 0.0;
  R->total = total;
  R->Z = total;
  R->edge_margin = 1.0;
  R->n_in = V;
  for (int64_t r = 0; r < V; ++r) {
    const double before = run;
    run += R->p[it[r].idx];
    R->in[it[r].idx] = 1;
    if (run >= cut || r == V - 1) {
      R->Z = run;
      R->n_in = r + 1;
      if (r < V - 1) {
        const double d1 = (run - cut) / total, d0 = (cut - before) / total;
        R->edge_margin = d1 < d0 ? d1 : d0;
      }
      break;
    }
  }
  free(it);
}

static int32_t orc_plain_draw(const orc_plain_row *R, uint32_t u24, double *margin) {
  const double target = ((double)u24 / 16777216.0) * R->Z;
  double run = 0.0, mg = R->edge_margin;
  int32_t tok = -1;
  int64_t last = -1;
  for (int64_t i = 0; i < R->V; ++i) {
    if (!R->in[i]) continue;
    last = i;
    const double before = run;
    run += R->p[i];
    if (run > target) {
      tok = (int32_t)i;
      const double d0 = (target - before) / R->total, d1 = (run - target) / R->total;
      if (d0 < mg) mg = d0;
      if (d1 < mg) mg = d1;
      break;
    }
  }
  if (tok < 0) { tok = (int32_t)last; mg = 0.0; }   /* rounding left the target at the very end: undecided */
  if (margin) *margin = mg;
  return tok;
}

int32_t orc_sample_plain(const float *logits, int64_t V, float temperature, float top_p, uint32_t u24, double *margin) {
  if (temperature <= 0.0f) {
    int64_t best = 0;
    for (int64_t i = 1; i < V; ++i)
      if (logits[i] > logits[best]) best = i;
    if (margin) *margin = 1.0;
    return (int32_t)best;
  }
  orc_plain_row R;
  orc_plain_prepare(&R, logits, V, temperature, top_p);
  const int32_t tok = orc_plain_draw(&R, u24, margin);
  free(R.p); free(R.in);
  return tok;
}

void orc_sample_plain_many(const float *logits, int64_t V, float temperature, float top_p, const uint32_t *u24, int64_t n,
                           int32_t *tokens, double *margins) {
  orc_plain_row R;
  orc_plain_prepare(&R, logits, V, temperature, top_p);
  for (int64_t k = 0; k < n; ++k) tokens[k] = orc_plain_draw(&R, u24[k], margins ? margins + k : NULL);
  free(R.p); free(R.in);
}

/* The integer specification (orc_sample) for n variates against one row: the same weights, cut and draw,
 * with the row sorted once.  temperature > 0. */
void orc_sample_many(const float *logits, int64_t V, float temperature, float top_p, const uint32_t *u24, int64_t n,
                     int32_t *tokens) {
  int64_t best = 0;
  for (int64_t i = 1; i < V; ++i)
    if (logits[i] > logits[best]) best = i;
  const float mx = logits[best];
  const float inv_t_log2e = 0x1.715476p+0f / temperature;
  uint64_t *wgt = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)V);
  orc_item *it = (orc_item *)malloc(sizeof(orc_item) * (size_t)V);
  uint64_t total = 0;
  for (int64_t i = 0; i < V; ++i) {
    wgt[i] = orc_weight(logits[i], mx, inv_t_log2e);
    total += wgt[i];
    it[i].idx = i;
    it[i].logit = logits[i];
  }
  qsort(it, (size_t)V, sizeof(orc_item), orc_item_desc);
  uint64_t cut = (uint64_t)floor((double)top_p * (double)total);
  if (cut > total) cut = total;
  char *in = (char *)calloc((size_t)V, 1);
  uint64_t run = 0, Z = 0;
  for (int64_t r = 0; r < V; ++r) {
    run += wgt[it[r].idx];
    in[it[r].idx] = 1;
    if (run >= cut) { Z = run; break; }
  }
  for (int64_t k = 0; k < n; ++k) {
    const unsigned __int128 prod = (unsigned __int128)u24[k] * (unsigned __int128)Z;
    const uint64_t rdraw = (uint64_t)(prod >> 24);
    int32_t tok = -1;
    uint64_t acc = 0;
    for (int64_t i = 0; i < V; ++i) {
      if (!in[i]) continue;
      acc += wgt[i];
      if (acc > rdraw) { tok = (int32_t)i; break; }
    }
    tokens[k] = tok;
  }
  free(wgt); free(it); free(in);
}

int orc_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp master
    n = omp_get_num_threads();
  }
#endif
  return n;
}
