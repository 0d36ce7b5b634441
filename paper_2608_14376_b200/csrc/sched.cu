// Host scheduler around a CoRun engine: the paper's isolated-prefill wrapper (Algorithms 1 and 2)
// with the wrapped scheduler reduced to "one decode iteration over every running request".
// Pure host code; the engine is reached through a table of callbacks.
#include <cstring>
#include <deque>
#include <new>
#include <vector>

#include "../../include/corun_sched.h"

namespace {

struct Request {
  std::vector<int32_t> prompt;
  std::vector<int32_t> out;       // tokens produced so far (the first comes from the prefill)
  int32_t max_new = 0;
  corun_sampling sampling{0.f, 1.f};
  uint64_t seed = 0;
  int32_t slot = -1;              // >= 0 while running
  bool finished = false;
};

}  // namespace

struct corun_sched {
  corun_sched_ops ops{};
  void *ctx = nullptr;
  int32_t B = 0, kv_block = 0, max_context = 0;
  std::vector<Request> reqs;             // by request id
  std::deque<int64_t> waiting;           // FIFO of request ids that have not started prefill
  std::vector<int64_t> running;          // request ids that own a slot; the most recently admitted first
  std::vector<int64_t> slot_owner;       // [B] request id or -1
  // scratch of a decode iteration
  std::vector<uint8_t> active;
  std::vector<uint64_t> seeds;
  std::vector<int32_t> toks;
};

namespace {

// Algorithm 1's second admission test ("can_fit_full_sequence"): pages for prompt + max_new tokens.
bool can_fit_full_sequence(corun_sched *s, const Request &r, int *status) {
  const int64_t need = ((int64_t)r.prompt.size() + r.max_new + s->kv_block - 1) / s->kv_block;
  const int64_t have = s->ops.free_blocks(s->ctx);
  if (have < 0) { *status = (int)have; return false; }
  return need <= have;
}

void finish(corun_sched *s, int64_t id) {
  Request &r = s->reqs[(size_t)id];
  r.finished = true;
  if (r.slot >= 0) s->slot_owner[(size_t)r.slot] = -1;
  r.slot = -1;
  for (size_t i = 0; i < s->running.size(); ++i)
    if (s->running[i] == id) { s->running.erase(s->running.begin() + (long)i); break; }
}

// Engine adapters for corun_sched_create_for_engine.
int eng_prefill(void *c, int32_t slot, const int32_t *t, int32_t n, int32_t reserve, const corun_sampling *sp, uint64_t seed,
                int32_t *first) {
  return corun_prefill((corun_engine *)c, slot, t, n, reserve, sp, seed, first);
}
int eng_decode(void *c, const uint8_t *a, const uint64_t *sd, int32_t *out) { return corun_decode_step((corun_engine *)c, a, sd, out); }
int eng_release(void *c, int32_t slot) { return corun_release((corun_engine *)c, slot); }
int64_t eng_free(void *c) { return corun_free_blocks((corun_engine *)c); }

}  // namespace

extern "C" int corun_sched_create(const corun_sched_ops *ops, void *ctx, int32_t B, int32_t kv_block, int32_t max_context,
                                  corun_sched **out) {
  if (!ops || !out || !ops->prefill || !ops->decode_step || !ops->release || !ops->free_blocks || B < 1 || kv_block < 1 ||
      max_context < 2)
    return CORUN_EINVAL;
  corun_sched *s = new (std::nothrow) corun_sched();
  if (!s) return CORUN_ENOMEM;
  s->ops = *ops;
  s->ctx = ctx;
  s->B = B;
  s->kv_block = kv_block;
  s->max_context = max_context;
  s->slot_owner.assign((size_t)B, -1);
  s->active.assign((size_t)B, 0);
  s->seeds.assign((size_t)B, 0);
  s->toks.assign((size_t)B, -1);
  *out = s;
  return CORUN_OK;
}

extern "C" int corun_sched_create_for_engine(corun_engine *e, corun_sched **out) {
  int32_t B = 0, max_context = 0, kv_block = 0;
  const int rc = corun_engine_info(e, &B, &max_context, &kv_block, nullptr);
  if (rc != CORUN_OK) return rc;
  const corun_sched_ops ops{eng_prefill, eng_decode, eng_release, eng_free};
  return corun_sched_create(&ops, e, B, kv_block, max_context, out);
}

extern "C" void corun_sched_destroy(corun_sched *s) { delete s; }

extern "C" int corun_sched_submit(corun_sched *s, const int32_t *prompt, int32_t n, int32_t max_new_tokens,
                                  const corun_sampling *sampling, uint64_t seed, int64_t *request_id) {
  if (!s || !prompt || !sampling || !request_id || n < 1 || max_new_tokens < 1 ||
      (int64_t)n + max_new_tokens > s->max_context)
    return CORUN_EINVAL;
  Request r;
  r.prompt.assign(prompt, prompt + n);
  r.max_new = max_new_tokens;
  r.sampling = *sampling;
  r.seed = seed;
  s->reqs.push_back(std::move(r));
  *request_id = (int64_t)s->reqs.size() - 1;
  s->waiting.push_back(*request_id);
  return CORUN_OK;
}

extern "C" int corun_sched_step(corun_sched *s, int32_t *action, int64_t *request_id, int32_t *n_active) {
  if (!s || !action || !request_id || !n_active) return CORUN_EINVAL;
  *action = CORUN_SCHED_IDLE;
  *request_id = -1;
  *n_active = 0;
  // ---- Algorithm 1: is there a request to prefill?  (A partly prefilled head of `running` cannot
  // exist here: a prefill runs all its chunks within one step.)
  if (!s->waiting.empty() && (int32_t)s->running.size() < s->B) {
    const int64_t id = s->waiting.front();
    Request &r = s->reqs[(size_t)id];
    int status = CORUN_OK;
    if (can_fit_full_sequence(s, r, &status)) {
      // ---- Algorithm 2: the selected request is the only one the engine sees in this iteration
      int32_t slot = -1;
      for (int32_t i = 0; i < s->B; ++i)
        if (s->slot_owner[(size_t)i] < 0) { slot = i; break; }
      if (slot < 0) return CORUN_ESLOT;   // cannot happen: running.size() < B
      int32_t first = -1;
      const int rc = s->ops.prefill(s->ctx, slot, r.prompt.data(), (int32_t)r.prompt.size(),
                                    (int32_t)r.prompt.size() + r.max_new, &r.sampling, r.seed, &first);
      if (rc != CORUN_OK) return rc;
      s->waiting.pop_front();
      r.slot = slot;
      s->slot_owner[(size_t)slot] = id;
      s->running.insert(s->running.begin(), id);   // Algorithm 2 puts the prefilled request in front of `running`
      r.out.push_back(first);
      *action = CORUN_SCHED_PREFILL;
      *request_id = id;
      *n_active = 1;
      if ((int32_t)r.out.size() >= r.max_new) {
        const int rr = s->ops.release(s->ctx, slot);
        finish(s, id);
        if (rr != CORUN_OK) return rr;
      }
      return CORUN_OK;
    }
    if (status != CORUN_OK) return status;
  }
  // ---- no prefill: a normal decode iteration over everything that runs
  if (s->running.empty()) return CORUN_OK;
  for (int32_t i = 0; i < s->B; ++i) {
    const int64_t id = s->slot_owner[(size_t)i];
    s->active[(size_t)i] = id >= 0 ? 1 : 0;
    s->seeds[(size_t)i] = id >= 0 ? s->reqs[(size_t)id].seed : 0;
  }
  const int rc = s->ops.decode_step(s->ctx, s->active.data(), s->seeds.data(), s->toks.data());
  if (rc != CORUN_OK) return rc;
  *action = CORUN_SCHED_DECODE;
  *n_active = (int32_t)s->running.size();
  int worst = CORUN_OK;
  for (int32_t i = 0; i < s->B; ++i) {
    const int64_t id = s->slot_owner[(size_t)i];
    if (id < 0) continue;
    Request &r = s->reqs[(size_t)id];
    r.out.push_back(s->toks[(size_t)i]);
    if ((int32_t)r.out.size() >= r.max_new) {
      const int rr = s->ops.release(s->ctx, i);
      finish(s, id);
      if (rr != CORUN_OK) worst = rr;
    }
  }
  return worst;
}

extern "C" int corun_sched_poll(corun_sched *s, int64_t request_id, int32_t *tokens, int32_t cap, int32_t *n_tokens,
                                int32_t *finished) {
  if (!s || request_id < 0 || request_id >= (int64_t)s->reqs.size() || cap < 0 || (cap > 0 && !tokens)) return CORUN_EINVAL;
  const Request &r = s->reqs[(size_t)request_id];
  const int32_t n = (int32_t)r.out.size();
  if (cap > 0 && n > 0) std::memcpy(tokens, r.out.data(), sizeof(int32_t) * (size_t)(n < cap ? n : cap));
  if (n_tokens) *n_tokens = n;
  if (finished) *finished = r.finished ? 1 : 0;
  return CORUN_OK;
}

extern "C" int corun_sched_slot_of(corun_sched *s, int64_t request_id, int32_t *slot) {
  if (!s || !slot || request_id < 0 || request_id >= (int64_t)s->reqs.size()) return CORUN_EINVAL;
  *slot = s->reqs[(size_t)request_id].slot;
  return CORUN_OK;
}

extern "C" int corun_sched_counts(corun_sched *s, int32_t *n_waiting, int32_t *n_running) {
  if (!s) return CORUN_EINVAL;
  if (n_waiting) *n_waiting = (int32_t)s->waiting.size();
  if (n_running) *n_running = (int32_t)s->running.size();
  return CORUN_OK;
}
