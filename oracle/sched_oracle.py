"""Plain restatement of the paper's isolated-prefill scheduling (Design, "Isolated Prefill":
Algorithm 1 "Finding the request for isolated prefill" and Algorithm 2 "Scheduling isolated prefill").

TEST INFRASTRUCTURE ONLY: imported by ``tests/``.  It shares no code with the library's scheduler
and never imports it.

The algorithms wrap an existing scheduler (``schedule_origin``).  Here that scheduler is the
smallest one that makes the wrapper meaningful, in the paper's vocabulary:

* two queues, ``running`` (requests that have started execution) and ``waiting`` (requests that
  have not started prefill);
* ``schedule_origin()`` first continues the prefill of every running request that still has
  prompt tokens to compute (one chunk of at most ``chunk`` tokens each), then admits waiting
  requests in order (first chunk each) while the running limit allows and the head's whole
  sequence fits -- the same two tests as Algorithm 1, so it never admits what Algorithm 1
  declined (by the paper, an iteration for which Algorithm 1 finds no request is an ordinary
  decode iteration; this is the reading of that statement) and it stops at the first request that
  does not fit.  Such requests form the iteration's prefill batch; if the batch is empty it
  schedules one decode token for every running request.  Left to itself it would batch several
  prefills together; Algorithm 2 hides all but one request from it.

Nothing here computes tokens: a request produces ``max_new`` tokens, the first at the end of its
prefill, and then leaves.  KV capacity is counted in pages of ``kv_block`` tokens; a request's
pages for its whole configured sequence (prompt + max_new) are taken when it is admitted
(Algorithm 1, "can_fit_full_sequence") and returned when it leaves, so nothing is ever preempted.
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class Request:
    rid: int
    num_prompt_tokens: int
    max_new: int
    num_computed_tokens: int = 0
    num_output_tokens: int = 0
    pages: int = 0


@dataclass
class Iteration:
    kind: str                       # "prefill" | "decode" | "idle"
    requests: list = field(default_factory=list)   # request ids taking part, in `running` order
    tokens: int = 0                 # prompt tokens computed (prefill) or 0


class Scheduler:
    def __init__(self, max_num_reqs: int, pool_pages: int, kv_block: int = 16, chunk: int = 256):
        self.max_num_reqs = max_num_reqs
        self.free_pages = pool_pages
        self.kv_block = kv_block
        self.chunk = chunk
        self.running: list[Request] = []
        self.waiting: list[Request] = []
        self.finished: list[int] = []
        self.failed: list[int] = []      # requests dropped because they can never fit the pool
        self._next = 0

    # ------------------------------------------------------------------ requests
    def add_request(self, num_prompt_tokens: int, max_new: int) -> int:
        r = Request(self._next, num_prompt_tokens, max_new)
        self._next += 1
        self.waiting.append(r)
        return r.rid

    def can_fit_full_sequence(self, r: Request) -> bool:
        need = -(-(r.num_prompt_tokens + r.max_new) // self.kv_block)
        return need <= self.free_pages

    # ------------------------------------------------------------------ which request gets an isolated prefill
    def isolated_prefill_candidate(self):
        """The paper's selection rule (Algorithm 1), from its prose: a request whose prompt is only partly
        computed is finished first (it can only be the one at the front of `running`, where the previous
        isolated prefill put it); otherwise the oldest waiting request is taken, provided the number of running
        requests is below the limit and the pool can hold its whole configured sequence.  None: no isolated
        prefill in this iteration."""
        partly = [r for r in self.running[:1] if r.num_computed_tokens < r.num_prompt_tokens]
        if partly:
            return partly[0]
        has_slot = len(self.running) < self.max_num_reqs
        if self.waiting and has_slot and self.can_fit_full_sequence(self.waiting[0]):
            return self.waiting[0]
        return None

    # ------------------------------------------------------------------ the wrapped scheduler
    def schedule_origin(self) -> Iteration:
        batch, tokens = [], 0
        for r in self.running:
            if r.num_computed_tokens < r.num_prompt_tokens:
                n = min(self.chunk, r.num_prompt_tokens - r.num_computed_tokens)
                r.num_computed_tokens += n
                batch.append(r); tokens += n
        while self.waiting and len(self.running) < self.max_num_reqs and self.can_fit_full_sequence(self.waiting[0]):
            r = self.waiting.pop(0)
            r.pages = -(-(r.num_prompt_tokens + r.max_new) // self.kv_block)
            self.free_pages -= r.pages
            n = min(self.chunk, r.num_prompt_tokens)
            r.num_computed_tokens = n
            self.running.append(r)
            batch.append(r); tokens += n
        if batch:
            it = Iteration("prefill", [r.rid for r in batch], tokens)
            for r in batch:
                if r.num_computed_tokens == r.num_prompt_tokens:
                    r.num_output_tokens = 1                   # the prefill's last position samples the first token
            self._retire()
            return it
        if not self.running:
            return Iteration("idle")
        it = Iteration("decode", [r.rid for r in self.running])
        for r in self.running:
            r.num_output_tokens += 1
        self._retire()
        return it

    def _retire(self):
        for r in list(self.running):
            if r.num_computed_tokens == r.num_prompt_tokens and r.num_output_tokens >= r.max_new:
                self.running.remove(r)
                self.free_pages += r.pages
                self.finished.append(r.rid)

    # ------------------------------------------------------------------ one iteration with the isolation wrapper
    def schedule(self) -> Iteration:
        """The paper's wrapper (Algorithm 2), from its prose: when a request was selected, the wrapped scheduler
        runs on a view of the queues that holds nothing but that request -- so it cannot batch anything with it
        -- and afterwards everything that was hidden is put back behind it in the order it had: the rest of
        `running` behind the request (which now runs), the rest of `waiting` untouched.  Without a selected
        request the wrapped scheduler sees the real queues (an ordinary decode iteration)."""
        chosen = self.isolated_prefill_candidate()
        if chosen is None:
            if not self.running and self.waiting:
                # nothing runs, the pool is all free, and the oldest request still does not fit: it never will;
                # it is dropped (reported as finished without tokens) so that the queue behind it can move
                dead = self.waiting.pop(0)
                self.finished.append(dead.rid)
                self.failed.append(dead.rid)
                return Iteration("idle", [dead.rid])
            return self.schedule_origin()
        was_running = any(r is chosen for r in self.running)
        hidden_running = [r for r in self.running if r is not chosen]
        hidden_waiting = [r for r in self.waiting if r is not chosen]
        self.running = [chosen] if was_running else []
        self.waiting = [] if was_running else [chosen]
        result = self.schedule_origin()
        self.running = self.running + hidden_running
        self.waiting = self.waiting + hidden_waiting
        return result

    # ------------------------------------------------------------------ one decision of the collapsed form
    def decision(self) -> Iteration:
        """``schedule()`` until the request it started prefilling has all its prompt computed: the
        chunks of one prefill as one record (Algorithm 1 resumes a partial prefill before anything
        else, so they are consecutive anyway)."""
        it = self.schedule()
        if it.kind != "prefill":
            return it
        rid = it.requests[0]
        while True:
            head = self.running[0] if self.running else None
            if head is None or head.rid != rid or head.num_computed_tokens >= head.num_prompt_tokens:
                return it
            nxt = self.schedule()
            assert nxt.kind == "prefill" and nxt.requests == [rid]
            it.tokens += nxt.tokens


# ---------------------------------------------------------------------------------------------------------
# Extension (not in the paper's algorithms): prefill requests batched with each other, the first direction
# of the paper's Future Work ("Batch-Invariant Kernels for Prefill").  The rule, stated once here and
# pinned by hand-derived traces (tests/golden/sched_batched_prefill_traces.txt):
#   a prefill decision takes the head of `waiting` exactly as Algorithm 1 does, then, in queue order, every
#   following request that still finds a slot, fits the pool together with those taken before it, and does
#   not add a chunk: each request's rows start on a multiple of `tile`, and ceil(rows / chunk) must stay what
#   it is without the request.  The first request that fails any of the three ends the batch.
def fill_batch(waiting, n_running: int, max_num_reqs: int, free_pages: int, kv_block: int, chunk: int, tile: int):
    """``waiting``: list of (num_prompt_tokens, max_new) in queue order, its head already admissible.
    Returns how many requests from the front are prefilled together (>= 1)."""
    pages = lambda r: -(-(r[0] + r[1]) // kv_block)
    chunks = lambda rows: -(-rows // chunk)
    taken, rows, used = 1, waiting[0][0], pages(waiting[0])
    for r in waiting[1:]:
        if n_running + taken >= max_num_reqs:
            break
        if used + pages(r) > free_pages:
            break
        start = -(-rows // tile) * tile
        if chunks(start + r[0]) != chunks(rows):
            break
        taken, rows, used = taken + 1, start + r[0], used + pages(r)
    return taken


class BatchedScheduler(Scheduler):
    """The collapsed scheduler (``decision``) with the extension: one record per batched prefill."""

    def __init__(self, max_num_reqs: int, pool_pages: int, kv_block: int = 16, chunk: int = 256, tile: int = 32):
        super().__init__(max_num_reqs, pool_pages, kv_block, chunk)
        self.tile = tile

    def decision(self) -> Iteration:
        det = self.isolated_prefill_candidate()
        if det is None or det in self.running:
            return super().decision()
        n = fill_batch([(r.num_prompt_tokens, r.max_new) for r in self.waiting], len(self.running), self.max_num_reqs,
                       self.free_pages, self.kv_block, self.chunk, self.tile)
        out = Iteration("prefill")
        for _ in range(n):                                    # each taken request is admitted as Algorithm 1 admits one
            it = super().decision()
            assert it.kind == "prefill" and len(it.requests) == 1
            out.requests += it.requests
            out.tokens += it.tokens
        return out
