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
  // batched prefill (off unless enabled)
  corun_sched_prefill_batch_fn prefill_batch = nullptr;
  int32_t chunk_rows = 0, tile_rows = 0;
  bool for_engine = false;
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
int eng_prefill_batch(void *c, int32_t n, const int32_t *slots, const int32_t *t, const int32_t *nt, const int32_t *res,
                      const corun_sampling *sp, const uint64_t *seeds, int32_t *first) {
  return corun_prefill_batch((corun_engine *)c, n, slots, t, nt, res, sp, seeds, first);
}

// After its prefill a request runs in `slot` with its first token; it may be finished already.
int admitted(corun_sched *s, int64_t id, int32_t slot, int32_t first) {
  Request &r = s->reqs[(size_t)id];
  r.slot = slot;
  s->slot_owner[(size_t)slot] = id;
  s->running.insert(s->running.begin(), id);   // Algorithm 2 puts the prefilled request in front of `running`
  r.out.push_back(first);
  if ((int32_t)r.out.size() >= r.max_new) {
    const int rr = s->ops.release(s->ctx, slot);
    finish(s, id);
    return rr;
  }
  return CORUN_OK;
}

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
  const int rc2 = corun_sched_create(&ops, e, B, kv_block, max_context, out);
  if (rc2 == CORUN_OK) (*out)->for_engine = true;
  return rc2;
}

extern "C" int corun_sched_enable_batched_prefill(corun_sched *s, corun_sched_prefill_batch_fn fn, int32_t chunk_rows,
                                                  int32_t tile_rows) {
  if (!s) return CORUN_EINVAL;
  if (!fn) {
    if (!s->for_engine) return CORUN_EINVAL;
    const int rc = corun_prefill_geometry((corun_engine *)s->ctx, &chunk_rows, &tile_rows);
    if (rc != CORUN_OK) return rc;
    fn = eng_prefill_batch;
  }
  if (tile_rows < 1 || chunk_rows < tile_rows || chunk_rows % tile_rows) return CORUN_EINVAL;
  s->prefill_batch = fn;
  s->chunk_rows = chunk_rows;
  s->tile_rows = tile_rows;
  return CORUN_OK;
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
      if (s->prefill_batch) {
        // ---- extension: the requests behind the head that fit into the padding of the head's chunks
        const int64_t free_pages = s->ops.free_blocks(s->ctx);
        if (free_pages < 0) return (int)free_pages;
        auto pages_of = [&](const Request &q) { return ((int64_t)q.prompt.size() + q.max_new + s->kv_block - 1) / s->kv_block; };
        auto chunks_of = [&](int64_t rows) { return (rows + s->chunk_rows - 1) / s->chunk_rows; };
        std::vector<int64_t> ids{id};
        int64_t rows = (int64_t)r.prompt.size(), pages = pages_of(r);
        for (size_t w = 1; w < s->waiting.size(); ++w) {
          const Request &q = s->reqs[(size_t)s->waiting[w]];
          if ((int32_t)(s->running.size() + ids.size()) >= s->B) break;
          if (pages + pages_of(q) > free_pages) break;
          const int64_t start = (rows + s->tile_rows - 1) / s->tile_rows * s->tile_rows;
          if (chunks_of(start + (int64_t)q.prompt.size()) != chunks_of(rows)) break;
          ids.push_back(s->waiting[w]);
          rows = start + (int64_t)q.prompt.size();
          pages += pages_of(q);
        }
        if (ids.size() > 1) {
          const int n = (int)ids.size();
          std::vector<int32_t> slots, toks, lens, res, first((size_t)n, -1);
          std::vector<corun_sampling> smp;
          std::vector<uint64_t> seeds;
          int32_t next = 0;
          for (int64_t q : ids) {
            const Request &rq = s->reqs[(size_t)q];
            while (next < s->B && s->slot_owner[(size_t)next] >= 0) ++next;
            if (next >= s->B) return CORUN_ESLOT;   // cannot happen: running + taken < B
            slots.push_back(next++);
            toks.insert(toks.end(), rq.prompt.begin(), rq.prompt.end());
            lens.push_back((int32_t)rq.prompt.size());
            res.push_back((int32_t)rq.prompt.size() + rq.max_new);
            smp.push_back(rq.sampling);
            seeds.push_back(rq.seed);
          }
          const int rc = s->prefill_batch(s->ctx, n, slots.data(), toks.data(), lens.data(), res.data(), smp.data(),
                                          seeds.data(), first.data());
          if (rc != CORUN_OK) return rc;
          int worst = CORUN_OK;
          for (int i = 0; i < n; ++i) {
            s->waiting.pop_front();
            const int rr = admitted(s, ids[(size_t)i], slots[(size_t)i], first[(size_t)i]);
            if (rr != CORUN_OK) worst = rr;
          }
          *action = CORUN_SCHED_PREFILL;
          *request_id = id;
          *n_active = n;
          return worst;
        }
      }
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
      *action = CORUN_SCHED_PREFILL;
      *request_id = id;
      *n_active = 1;
      return admitted(s, id, slot, first);
    }
    if (status != CORUN_OK) return status;
    if (s->running.empty()) {
      // Nothing runs, so every page the pool has is free, and the head still does not fit: it never will.
      // Left in place it would block the queue for good (nothing overtakes the head): the request fails.
      s->waiting.pop_front();
      r.finished = true;
      *request_id = id;
      return CORUN_ENOSPACE;
    }
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
