/*
 * corun.h -- C ABI of the CoRun hot path for NVIDIA B200 (sm_100a).
 *
 * One engine = one GPU, one model, ONE fixed padded decode shape (B slots,
 * max_context).  A request lives in a slot: corun_prefill runs its prompt alone
 * (batch of one, natural length, fixed-size chunks) and fills the slot's paged
 * KV cache; corun_decode_step runs one fixed-shape decode iteration over all B
 * slots, with padding in the unused ones, as a single CUDA-graph replay.
 *
 * Guarantee (paper, Design, "Determinism Contract" and "Determinism Argument"):
 * within one engine the logits and tokens of a request are bitwise identical
 * whatever slot it occupies, whatever requests or padding occupy the other
 * slots, and across repeated runs.  Nothing is promised across different B,
 * max_context, GPUs or library builds (same section, non-claims).
 *
 * Conventions
 *   - every function returns 0 (CORUN_OK) or a negative corun_status; nothing
 *     aborts, throws or traps;
 *   - "device" pointers are CUDA device memory of the current device, "host"
 *     pointers ordinary host memory;
 *   - weight memory is BORROWED: allocated by the caller, never written, and it
 *     must outlive the engine.  Everything else (KV pool, block tables,
 *     workspaces, logits, the graph) is owned by the engine;
 *   - host arrays are read/written only during the call; calls are synchronous
 *     unless stated otherwise; an engine is not thread-safe;
 *   - all kernels run on the stream given to corun_init.
 */
#ifndef CORUN_H_
#define CORUN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CORUN_OK = 0,
  CORUN_EINVAL = -1,   /* NULL pointer, bad shape, bad argument                         */
  CORUN_ESLOT = -2,    /* slot out of range; busy on prefill; empty on decode / release */
  CORUN_ENOSPACE = -3, /* the KV pool cannot hold the request's full reserved sequence  */
  CORUN_ECTX = -4,     /* an active slot would exceed its reserved length               */
  CORUN_ECUDA = -5,    /* a CUDA call failed (corun_last_cuda_error has the code)       */
  CORUN_ETIMEOUT = -6, /* a bounded device-side wait expired (device status word)       */
  CORUN_ENOMEM = -7,   /* device or host allocation failed                              */
  CORUN_ELIMIT = -8    /* a size exceeds the fixed capacity of corun_gemm_static        */
} corun_status;

typedef struct corun_engine corun_engine; /* opaque, owned by the library */

/* Decoder shape.  arch 0 = dense GQA decoder: pre-norm RMSNorm, half-split
 * RoPE on q and k, causal softmax attention, SwiGLU FFN, untied LM head, no
 * biases.  Requirements: hidden, ffn and n_q_heads*head_dim multiples of 64;
 * head_dim 64 or 128; n_q_heads / n_kv_heads in {1,2,4,8}.  arch 1 = decoder with multi-head latent
 * attention: accepted by corun_init_mla only (which takes 0 as well and ignores n_kv_heads and head_dim). */
typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  float rms_eps, rope_theta;
  int32_t arch;
} corun_shape;

/* Device pointers to bf16 weights, row-major [out_features, in_features].
 *   embed [vocab, hidden]; lm_head [vocab, hidden]; final_norm [hidden];
 *   per layer (arrays of n_layers device pointers, the arrays themselves on the host):
 *   attn_norm [hidden]; wqkv [(nq+2nkv)*hd, hidden] (q rows, then k, then v);
 *   wo [hidden, nq*hd]; mlp_norm [hidden]; wgate_up [2*ffn, hidden] (gate rows,
 *   then up rows); wdown [hidden, ffn].
 * Matrix base addresses must be 16-byte aligned. */
typedef struct {
  const void *embed, *lm_head, *final_norm;
  const void *const *attn_norm, *const *wqkv, *const *wo;
  const void *const *mlp_norm, *const *wgate_up, *const *wdown;
} corun_weights;

/* temperature <= 0 selects greedy argmax (lowest id on ties); otherwise
 * temperature -> softmax -> top-p nucleus -> inverse CDF (see corun_decode_step). */
typedef struct {
  float temperature, top_p;
} corun_sampling;

/*
 * Creates an engine for the fixed decode shape (B, max_context) and captures
 * its decode graph (paper, Design, "Fixed-Shape Batched Decode": one captured
 * shape equal to the maximum concurrency, replayed for every decode iteration).
 *   B               1..256 slots.
 *   max_context     largest prompt + generated length of any request.
 *   kv_block        tokens per KV page; must be 16.
 *   kv_pool_blocks  pages in the pool; 0 = B * ceil(max_context / kv_block), or as many as fit in the
 *                   device memory that is free now less 6 GiB, whichever is less.
 *   cuda_stream     a cudaStream_t (NULL = the legacy default stream).
 * Errors: EINVAL, ENOMEM, ECUDA.  On success *out owns device memory until
 * corun_destroy.
 */
int corun_init(const corun_shape *shape, const corun_weights *weights, int32_t B, int32_t max_context,
               int32_t kv_block, int64_t kv_pool_blocks, void *cuda_stream, corun_engine **out);

/*
 * The same engine with Mixture-of-Experts feed-forward layers (the paper's evaluated models are MoE
 * decoders -- Evaluation, "Setup"): grouped-query attention as above, every feed-forward layer a
 * router + routed experts (+ always-on shared experts) computed without expert groups, so that a row's
 * result does not depend on which rows share the step (include/corun_moe.h describes the block).
 * shape->ffn and weights->wgate_up / wdown are ignored (the arrays may be NULL).
 *   router   L device pointers, bf16 [E, H]
 *   gate_up  L device pointers, bf16 [(E + n_shared) * 2F, H]: block e = expert e, gate rows then up rows;
 *            shared experts behind the routed ones
 *   down     L device pointers, bf16 [H, (E + n_shared) * F]: columns e*F.. of expert e
 * n_experts 1..256, top_k 1..min(E, 16), expert_ffn a multiple of 64; renormalize: the selected
 * probabilities divided by their sum.  Errors as corun_init.
 */
typedef struct {
  int32_t n_experts, top_k, expert_ffn, n_shared, renormalize;
  const void *const *router, *const *gate_up, *const *down;
} corun_moe_layers;
int corun_init_moe(const corun_shape *shape, const corun_weights *weights, const corun_moe_layers *moe, int32_t B,
                   int32_t max_context, int32_t kv_block, int64_t kv_pool_blocks, void *cuda_stream,
                   corun_engine **out);

/*
 * The same engine for a decoder with multi-head latent attention (MLA) -- the paper evaluates one MLA /
 * Mixture-of-Experts model (Evaluation, "Setup") -- at decode time in the absorbed form over a paged cache of
 * one latent vector and one shared rotary key per token (include/corun_mla.h describes the attention):
 *   [q | kv_a] = W_qkv RMSNorm(h):   q  = n_q_heads x [qk_nope | qk_rope],   kv_a = [kv_lora_rank | qk_rope]
 *   cached per token (fp16):  c = RMSNorm(kv_a[:rank]) * kv_norm,  r = RoPE(kv_a[rank:]) (half-split rotation)
 *   per head h, W_kv_b's block h = [W_uk (qk_nope rows) ; W_uv (v_head rows)] x rank:
 *     q_lat = W_uk^T q_nope,  s_t = (q_lat . c_t + RoPE(q_rope) . r_t) / sqrt(qk_nope + qk_rope),
 *     o_h = W_uv sum_t softmax(s)_t c_t;    y = W_o [o_0 | o_1 | ...]
 * shape->n_q_heads heads (at most 16); shape->n_kv_heads and shape->head_dim are ignored.  Weights as in
 * corun_weights except  wqkv [n_q_heads * (qk_nope + qk_rope) + rank + qk_rope, hidden]  and
 * wo [hidden, n_q_heads * v_head].  Layers 0 .. first_dense-1 have the dense SwiGLU feed-forward of width
 * shape->ffn (weights->wgate_up / wdown, entries of the other layers unused); the other layers are
 * Mixture-of-Experts layers as in corun_init_moe (entries of moe's arrays below first_dense unused).  moe may
 * be NULL when first_dense == n_layers.
 *   kv_norm  L device pointers, bf16 [rank]          wkv_b  L device pointers, bf16 [n_q_heads * (qk_nope + v_head), rank]
 * kv_lora_rank 256 or 512; qk_nope a multiple of 64; qk_rope even, a multiple of 8, at most 64;
 * qk_nope + v_head a multiple of 256; n_q_heads * v_head a multiple of 64.  A decode step of B slots and a
 * prefill chunk run the same kernels; a prefill row attends to its request's cache up to its own position.
 * kv_block may be 16 or 64 here: with 64 a slot's cache grows in blocks of 64 tokens (four pages of 16 tokens that
 * are neighbours in the pool, which the attention kernel fetches with one TMA box instead of four); kv_pool_blocks,
 * corun_free_blocks and corun_engine_info then count blocks of 64 tokens.  No value depends on the choice.
 * Errors as corun_init.
 */
typedef struct {
  int32_t kv_lora_rank, qk_nope, qk_rope, v_head, first_dense;
  const void *const *kv_norm, *const *wkv_b;
} corun_mla_layers;
int corun_init_mla(const corun_shape *shape, const corun_weights *weights, const corun_mla_layers *mla,
                   const corun_moe_layers *moe, int32_t B, int32_t max_context, int32_t kv_block, int64_t kv_pool_blocks,
                   void *cuda_stream, corun_engine **out);

/*
 * Isolated prefill (paper, Design, "Isolated Prefill"; Algorithm 1's admission
 * rule): runs the n prompt tokens of one request alone, in fixed-size chunks
 * whose sequence depends on n only, writes its KV cache, samples the first
 * token with R(seed, 0) from the last position's logits ("Shape-Aligned
 * Sampling": prefill presents one sampling row) and leaves that token pending
 * for the slot's first decode step.
 *   tokens       host, n ids in [0, vocab).
 *   reserve_len  prompt + maximum new tokens, <= max_context; pages for the
 *                whole reserved sequence are taken now, so a later decode step
 *                can never run out (no preemption, no recompute).
 *   out_first_token  host, may be NULL.
 * Errors: EINVAL; ESLOT (slot busy / out of range); ENOSPACE (reservation does
 * not fit; the engine is unchanged); ECUDA; ETIMEOUT.
 */
int corun_prefill(corun_engine *e, int32_t slot, const int32_t *tokens, int32_t n, int32_t reserve_len,
                  const corun_sampling *sampling, uint64_t seed, int32_t *out_first_token);

/*
 * Prefill of several requests in shared chunks (paper, Future Work, "Batch-
 * Invariant Kernels for Prefill": prefill requests batched with other prefill
 * requests, never with decode).  The prompts go through the same fixed-shape
 * prefill program as corun_prefill; the rows of a chunk are dealt in request
 * order, every piece of a request starting on a boundary of the attention
 * kernel's query tiles, so that short prompts share a chunk instead of padding
 * one each.  All kernels of the program are position-invariant in the chunk
 * and attention reads every key from the cache, so each request's cache,
 * logits and first token are bitwise those of corun_prefill on it alone.
 *   slots, n_tokens, reserve_lens, samplings, seeds   host, n_req entries
 *                (slots distinct and free).
 *   tokens       host, the prompts one after the other (sum of n_tokens ids).
 *   out_first_tokens  host, n_req entries, may be NULL.
 * Errors as corun_prefill; ENOSPACE if the reservations do not all fit (the
 * engine is unchanged).
 */
int corun_prefill_batch(corun_engine *e, int32_t n_req, const int32_t *slots, const int32_t *tokens,
                        const int32_t *n_tokens, const int32_t *reserve_lens, const corun_sampling *samplings,
                        const uint64_t *seeds, int32_t *out_first_tokens);

/*
 * One fixed-shape decode iteration (paper, Design, "Fixed-Shape Batched
 * Decode", "Shape-Aligned Sampling", "Determinism Argument"): every slot with
 * active[s] != 0 feeds its pending token at position = its context length,
 * appends K/V, attends over its own pages with a split count and combine order
 * that depend on its own length only, and samples token = S(logits, R(seeds[s], t_s))
 * where t_s counts the tokens this request has sampled so far (prefill used
 * t = 0).  Inactive and empty slots are padding: they run through the same
 * launch shape, consume no random variate, change no state and report -1.
 *   active      host, B bytes.       seeds  host, B values (read where active).
 *   out_tokens  host, B ints.
 * Sampling: weight_i = floor(2^40 * exp2(fl32(fl32(logit_i - max) * fl32(log2(e)/T))))
 * where exp2 is evaluated in fp32 as: n = rint(x), f = x - n, degree-7 Taylor
 * polynomial of 2^f (coefficients ln(2)^k/k! rounded to fp32) in Horner form with
 * separately rounded multiply and add, scaled exactly by 2^n -- an integer that is
 * identical on every IEEE-754 implementation; nucleus = tokens
 * by descending logit (ties: lower id first) up to and including the first
 * whose running weight reaches floor(top_p * total); draw r = floor(u24 * Z / 2^24)
 * with u24 the top 24 bits of Philox4x32-10(key = seed, counter = (t,0,0,0));
 * the token is the first nucleus member in ascending id order whose running
 * weight exceeds r.
 * Errors: EINVAL; ESLOT (an active slot is empty); ECTX (an active slot is at
 * its reserved length: the whole step is refused and nothing changes); ECUDA;
 * ETIMEOUT.
 */
int corun_decode_step(corun_engine *e, const uint8_t *active, const uint64_t *seeds, int32_t *out_tokens);

/* Asynchronous form for back-to-back replays: stages active/seeds and enqueues
 * one decode iteration on the engine's stream without waiting.  Results of the
 * last enqueued step are fetched by corun_decode_wait (out_tokens host, B ints,
 * may be NULL).  Same semantics and errors as corun_decode_step. */
int corun_decode_enqueue(corun_engine *e, const uint8_t *active, const uint64_t *seeds);
int corun_decode_wait(corun_engine *e, int32_t *out_tokens);

/* Frees the slot's pages and clears its state (host only).  ESLOT if empty. */
int corun_release(corun_engine *e, int32_t slot);

/* Destroys the engine and frees what it owns.  NULL is allowed. */
void corun_destroy(corun_engine *e);

/* ---- accessors used by tests and reports ---- */

/* Logits row (vocab floats, host) of the slot's latest forward pass: its prefill's until the slot takes part in a
 * decode step (other slots' steps in between leave them alone), then those of the last decode step it took part in,
 * readable until the next decode step (whose rows overwrite them). */
int corun_get_logits(corun_engine *e, int32_t slot, float *out);
/* Replaces the slot's pending token (teacher forcing). */
int corun_force_token(corun_engine *e, int32_t slot, int32_t token);
/* Cached tokens of the slot, or a negative status. */
int corun_context_len(corun_engine *e, int32_t slot);
/* Free pages left in the pool, or a negative status. */
int64_t corun_free_blocks(corun_engine *e);
/* The engine's fixed dimensions: slots, largest context, tokens per page, pages in the pool
 * (any of the out pointers may be NULL). */
int corun_engine_info(corun_engine *e, int32_t *B, int32_t *max_context, int32_t *kv_block, int64_t *pool_blocks);
/* How corun_prefill_batch packs prompts: rows per prefill chunk, and the row granularity on which every
 * piece of a request starts (the query tile of the prefill attention kernel).  Either pointer may be NULL. */
int corun_prefill_geometry(corun_engine *e, int32_t *chunk_rows, int32_t *tile_rows);
/* Number of kernel launches in one decode iteration. */
int corun_decode_launches(corun_engine *e);
/* Test and measurement accessors (cache read / write, adopting a slot without a prefill, eager launches,
 * per-kernel timing, the stand-alone GEMM and sampler, kernel timelines) are declared in corun_debug.h. */

/*
 * corun_gemm_static -- the stand-alone GEMM (corun_debug_gemm of corun_debug.h) for callers that cannot allocate.
 * (The paper has no counterpart; this is a service entry point of the library.)
 *
 * Same operation and argument meaning as corun_debug_gemm:
 *   out[r, n] = sum_k W[n, k] * X[r, k],  W bf16 [N, K], X fp32 [R, K], out fp32 [R, N],
 * all three in device memory owned by the caller.  It is meant for hosts that
 * may not call cudaMalloc where they need the product: code running inside an
 * arena that took all device memory at start-up, loops that cannot afford the
 * device-wide synchronisation an allocation or a free implies, processes with
 * a fixed memory budget.  Everything the kernel needs besides its inputs and
 * output (split activations, per-CTA partial sums, partition tables, status
 * word) lives in one array of about 6.3 MiB that is part of the library image:
 * every GPU that loads the library holds it until the process exits.
 *
 * Limits (fixed by that array): R <= CORUN_STATIC_MAX_ROWS, K <= CORUN_STATIC_MAX_K
 * (and K % 64 == 0), N <= CORUN_STATIC_MAX_N, at most 192 SMs.  Beyond them the
 * call returns CORUN_ELIMIT and does nothing.  The call makes no cudaMalloc,
 * cudaFree or any other allocating call.
 *
 * `out` and `W` must start on a 16-byte boundary (the kernels store and load
 * 16 bytes at a time), `X` on a 4-byte one; otherwise CORUN_EINVAL, before
 * anything is launched.
 *
 * The first call on each device resolves the array's device address and sets a
 * kernel attribute (safe from several host threads); that first call should come
 * before any stream capture.  Every call is synchronous on `cuda_stream`: it ends
 * with a stream synchronisation and a copy of the kernel's status word to the
 * host, so a call made while `cuda_stream` is capturing is refused with
 * CORUN_EINVAL.  All calls share the one array, which keeps the previous call's
 * contents (the call clears the parts that must start at zero): two calls that
 * overlap on the GPU -- from two threads, or on two streams -- race on it.
 * Errors: EINVAL, ELIMIT, ECUDA, ETIMEOUT.
 */
#define CORUN_STATIC_MAX_ROWS 16
#define CORUN_STATIC_MAX_K 4096
#define CORUN_STATIC_MAX_N 8192
int corun_gemm_static(const void *W, int32_t N, int32_t K, const float *X, int32_t R, float *out, void *cuda_stream);

const char *corun_strerror(int status);
int corun_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CORUN_H_ */
