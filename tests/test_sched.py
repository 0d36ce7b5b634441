"""Host scheduling (isolated prefill in front of the padded decode iteration).

The oracle (``oracle/sched_oracle.py``, Algorithms 1 and 2 written out) is pinned to hand-derived
iteration sequences and to the properties the paper states; the library's scheduler is then driven
against a stand-in engine (callbacks that only count pages) and must take the same decisions."""
import ctypes as C
import os

import numpy as np
import pytest

from oracle import sched_oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _golden_cases():
    cases, cur = [], None
    for line in open(os.path.join(ROOT, "tests", "golden", "sched_isolated_prefill_traces.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "case":
            cur = dict(name=t[1], reqs=[], its=[], **{k: int(v) for k, v in (x.split("=") for x in t[2:])})
            cases.append(cur)
        elif t[0] == "req":
            cur["reqs"].append((int(t[1]), int(t[2])))
        elif t[0] == "P":
            cur["its"].append(("prefill", [int(t[1])], int(t[2])))
        elif t[0] == "D":
            cur["its"].append(("decode", [int(x) for x in t[1:]], 0))
        elif t[0] == "I":
            cur["its"].append(("idle", [], 0))
    return cases


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
def test_oracle_reproduces_hand_derived_iterations(case):
    s = sched_oracle.Scheduler(case["max_num_reqs"], case["pool_pages"], case["kv_block"], case["chunk"])
    for p, m in case["reqs"]:
        s.add_request(p, m)
    got = []
    for _ in case["its"]:
        it = s.schedule()
        got.append((it.kind, it.requests, it.tokens))
    assert got == case["its"]
    assert s.free_pages == case["pool_pages"] and not s.running and not s.waiting


def _random_trace(seed, n_req=40):
    rng = np.random.default_rng(seed)
    B = int(rng.integers(1, 6))
    kv_block = 16
    reqs = [(int(rng.integers(1, 200)), int(rng.integers(1, 12))) for _ in range(n_req)]
    biggest = max(-(-(p + m) // kv_block) for p, m in reqs)
    pool = biggest + int(rng.integers(0, 3 * biggest))          # every request fits alone; often not together
    # submissions interleaved with decisions: ("submit", k) / ("step", k)
    script, left = [], n_req
    while left:
        k = int(min(left, rng.integers(1, 6)))
        script.append(("submit", k)); left -= k
        script.append(("step", int(rng.integers(0, 8))))
    return B, kv_block, pool, reqs, script


@pytest.mark.parametrize("seed", range(6))
def test_oracle_keeps_the_papers_properties(seed):
    B, kv_block, pool, reqs, script = _random_trace(seed)
    s = sched_oracle.Scheduler(B, pool, kv_block, chunk=64)
    its, nxt = [], 0
    for op, k in script + [("step", 10 ** 6)]:
        if op == "submit":
            for p, m in reqs[nxt:nxt + k]:
                s.add_request(p, m)
            nxt += k
            continue
        for _ in range(k):
            free_before, running_before = s.free_pages, [r.rid for r in s.running]
            waiting_before = [r.rid for r in s.waiting]
            it = s.schedule()
            its.append(it)
            if it.kind == "prefill":
                assert len(it.requests) == 1                      # a prefill batch is one request
                rid = it.requests[0]
                if rid in waiting_before:                         # admission: FIFO head, room for a slot and for the whole sequence
                    assert rid == waiting_before[0]
                    assert len(running_before) < B
                    assert -(-(sum(reqs[rid])) // kv_block) <= free_before
                else:                                             # continuing a chunked prefill: it was the head of running
                    assert rid == running_before[0]
            elif it.kind == "decode":
                assert it.requests == running_before              # everything that runs takes part: nothing is preempted
                head = waiting_before[0] if waiting_before else None
                assert head is None or len(running_before) >= B or -(-(sum(reqs[head])) // kv_block) > free_before
            else:
                assert not running_before
                if nxt == len(reqs) and not waiting_before:
                    break
            assert 0 <= s.free_pages <= pool and len(s.running) <= B
    # every request was prefilled exactly once over consecutive iterations, in submission order
    order, seen = [], {}
    for i, it in enumerate(its):
        if it.kind == "prefill":
            rid = it.requests[0]
            if rid in seen:
                assert seen[rid][-1] == i - 1                     # chunks of one prefill are not interrupted
            else:
                order.append(rid)
            seen.setdefault(rid, []).append(i)
    assert order == list(range(len(reqs)))
    assert {r: sum(its[i].tokens for i in ix) for r, ix in seen.items()} == {r: reqs[r][0] for r in range(len(reqs))}
    assert sorted(s.finished) == list(range(len(reqs))) and s.free_pages == pool
    # tokens per request: one from the prefill plus one per decode iteration it took part in
    for rid, (p, m) in enumerate(reqs):
        assert 1 + sum(1 for it in its if it.kind == "decode" and rid in it.requests) == m


class _StandInEngine:
    """Counts pages like the engine's admission does and records every call."""

    def __init__(self, B, pool, kv_block):
        from paper_2608_14376_b200 import corun

        self.corun, self.B, self.free, self.kv_block = corun, B, pool, kv_block
        self.pages = {}
        self.calls = []
        self.step_of = {}
        self.fail_next = None
        self.ops = corun.SchedOps(corun.PREFILL_FN(self._prefill), corun.DECODE_FN(self._decode),
                                  corun.RELEASE_FN(self._release), corun.FREE_BLOCKS_FN(lambda ctx: self.free))

    def _prefill(self, ctx, slot, tokens, n, reserve, sampling, seed, first):
        if self.fail_next == "prefill":
            self.fail_next = None
            return self.corun.ECUDA
        need = -(-reserve // self.kv_block)
        if slot in self.pages:
            return self.corun.ESLOT
        if need > self.free:
            return self.corun.ENOSPACE
        self.free -= need
        self.pages[slot] = need
        self.step_of[slot] = 1
        self.calls.append(("prefill", slot, n, reserve, int(seed)))
        first[0] = int(seed) % 1000
        return 0

    def _decode(self, ctx, active, seeds, out):
        if self.fail_next == "decode":
            self.fail_next = None
            return self.corun.ETIMEOUT
        act = [i for i in range(self.B) if active[i]]
        assert all(s in self.pages for s in act)
        for i in range(self.B):
            out[i] = (int(seeds[i]) % 1000 + self.step_of[i]) if active[i] else -1
            if active[i]:
                self.step_of[i] += 1
        self.calls.append(("decode", tuple(act), tuple(int(seeds[i]) for i in act)))
        return 0

    def _release(self, ctx, slot):
        self.free += self.pages.pop(slot)
        self.calls.append(("release", slot))
        return 0


@pytest.mark.parametrize("seed", range(6))
def test_library_scheduler_takes_the_oracles_decisions(seed):
    from paper_2608_14376_b200 import build, corun

    build.build()
    B, kv_block, pool, reqs, script = _random_trace(100 + seed)
    eng = _StandInEngine(B, pool, kv_block)
    sch = corun.Scheduler(ops=eng.ops, B=B, kv_block=kv_block, max_context=256)
    ref = sched_oracle.Scheduler(B, pool, kv_block, chunk=64)
    nxt, rid_of = 0, []
    try:
        for op, k in script + [("step", 10 ** 6)]:
            if op == "submit":
                for p, m in reqs[nxt:nxt + k]:
                    rid_of.append(sch.submit(np.arange(p) % 97, m, 0.7, 0.9, seed=5000 + len(rid_of)))
                    ref.add_request(p, m)
                nxt += k
                continue
            for _ in range(k):
                want = ref.decision()
                action, rid, n = sch.step()
                assert action == {"idle": corun.SCHED_IDLE, "prefill": corun.SCHED_PREFILL, "decode": corun.SCHED_DECODE}[want.kind]
                if want.kind == "prefill":
                    assert rid == want.requests[0] and n == 1
                    kind, slot, n_tok, reserve, sd = eng.calls[-1] if eng.calls[-1][0] == "prefill" else eng.calls[-2]
                    assert (kind, n_tok, reserve, sd) == ("prefill", reqs[rid][0], sum(reqs[rid]), 5000 + rid)
                elif want.kind == "decode":
                    assert n == len(want.requests)
                    dec = [c for c in eng.calls if c[0] == "decode"][-1]
                    assert sorted(dec[2]) == sorted(5000 + r for r in want.requests)   # exactly the running requests, with their own seeds
                assert sch.counts() == (len(ref.waiting), len(ref.running))
                assert eng.free == ref.free_pages
                if want.kind == "idle" and nxt == len(reqs):
                    break
        assert rid_of == list(range(len(reqs)))
        for rid, (p, m) in enumerate(reqs):
            toks, fin = sch.poll(rid)
            assert fin and len(toks) == m and sch.slot_of(rid) == -1
            assert list(toks) == [(5000 + rid) % 1000 + t for t in range(m)]   # the stand-in's tokens count the request's own steps
        assert eng.free == pool and not eng.pages
    finally:
        sch.close()


def test_library_scheduler_argument_and_engine_errors():
    from paper_2608_14376_b200 import build, corun

    build.build()
    L = corun.lib()
    h = C.c_void_p()
    assert L.corun_sched_create(None, None, 4, 16, 128, C.byref(h)) == corun.EINVAL
    assert L.corun_sched_create_for_engine(None, C.byref(h)) == corun.EINVAL
    assert L.corun_sched_step(None, None, None, None) == corun.EINVAL
    eng = _StandInEngine(2, 8, 16)
    sch = corun.Scheduler(ops=eng.ops, B=2, kv_block=16, max_context=64)
    try:
        with pytest.raises(corun.CorunError):
            sch.submit(np.zeros(60, np.int32), 10)          # longer than max_context
        with pytest.raises(corun.CorunError):
            sch.submit(np.zeros(0, np.int32), 1)
        with pytest.raises(corun.CorunError):
            sch.poll(0)
        a = sch.submit(np.zeros(10, np.int32), 3, seed=1)
        eng.fail_next = "prefill"
        with pytest.raises(corun.CorunError) as ei:
            sch.step()
        assert ei.value.status == corun.ECUDA and sch.counts() == (1, 0)      # nothing moved
        assert sch.step()[:2] == (corun.SCHED_PREFILL, a)
        eng.fail_next = "decode"
        with pytest.raises(corun.CorunError) as ei:
            sch.step()
        assert ei.value.status == corun.ETIMEOUT and sch.counts() == (0, 1) and len(sch.poll(a)[0]) == 1
        assert sch.step()[0] == corun.SCHED_DECODE and len(sch.poll(a)[0]) == 2
    finally:
        sch.close()


def test_a_request_that_can_never_fit_is_failed_and_the_queue_moves_on():
    """The pool holds 8 pages.  A request of 9 pages at the head of `waiting` can never be admitted: with
    nothing running the whole pool is free already.  Oracle and library drop it (finished, no tokens,
    ENOSPACE from the step) and serve the request behind it; while something runs the head only waits."""
    from paper_2608_14376_b200 import build, corun

    build.build()
    B, kv_block, pool = 2, 16, 8
    eng = _StandInEngine(B, pool, kv_block)
    sch = corun.Scheduler(ops=eng.ops, B=B, kv_block=kv_block, max_context=256)
    ref = sched_oracle.Scheduler(B, pool, kv_block, chunk=64)
    try:
        reqs = [(40, 3), (100, 40), (20, 2)]          # 3 pages, 9 pages (never fits), 2 pages
        ids = [sch.submit(np.arange(p) % 97, m, 0.7, 0.9, seed=7000 + i) for i, (p, m) in enumerate(reqs)]
        for p, m in reqs:
            ref.add_request(p, m)
        kinds, failed_at = [], None
        for i in range(12):
            want = ref.decision()
            try:
                action, rid, n = sch.step()
                assert want.kind != "idle" or not want.requests
                assert action == {"idle": corun.SCHED_IDLE, "prefill": corun.SCHED_PREFILL, "decode": corun.SCHED_DECODE}[want.kind]
            except corun.CorunError as e:
                assert e.status == corun.ENOSPACE and want.kind == "idle" and want.requests == [ids[1]]
                failed_at = i
            kinds.append(want.kind)
            assert sch.counts() == (len(ref.waiting), len(ref.running))
        # request 0 is served first (the big one waits behind it while it runs), then the big one is dropped,
        # then request 2 is served
        assert kinds[:3] == ["prefill", "decode", "decode"] and failed_at == 3 and kinds[4:6] == ["prefill", "decode"]
        assert ref.failed == [ids[1]]
        toks, fin = sch.poll(ids[1])
        assert fin and len(toks) == 0
        for i in (0, 2):
            toks, fin = sch.poll(ids[i])
            assert fin and len(toks) == reqs[i][1]
        assert eng.free == pool
    finally:
        sch.close()


# ------------------------------------------------------------------------------------------------ batched prefill
def _batched_cases():
    cases, cur = [], None
    for line in open(os.path.join(ROOT, "tests", "golden", "sched_batched_prefill_traces.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "case":
            cur = dict(name=t[1], reqs=[], its=[], **{k: int(v) for k, v in (x.split("=") for x in t[2:])})
            cases.append(cur)
        elif t[0] == "req":
            cur["reqs"].append((int(t[1]), int(t[2])))
        elif t[0] == "P":
            cut = t.index(":")
            cur["its"].append(("prefill", [int(x) for x in t[1:cut]], int(t[cut + 1])))
        elif t[0] == "D":
            cur["its"].append(("decode", [int(x) for x in t[1:]], 0))
        elif t[0] == "I":
            cur["its"].append(("idle", [], 0))
    return cases


@pytest.mark.parametrize("case", _batched_cases(), ids=lambda c: c["name"])
def test_batched_oracle_reproduces_hand_derived_decisions(case):
    s = sched_oracle.BatchedScheduler(case["max_num_reqs"], case["pool_pages"], case["kv_block"], case["chunk"], case["tile"])
    for p, m in case["reqs"]:
        s.add_request(p, m)
    got = []
    for _ in case["its"]:
        it = s.decision()
        got.append((it.kind, it.requests, it.tokens))
    assert got == case["its"]


@pytest.mark.parametrize("seed", range(6))
def test_batched_rule_properties(seed):
    """A batch is a prefix of the queue, never needs more chunks than its head alone, never more slots or
    pages than there are; and every request is served exactly as under the isolated policy (same number of
    tokens, nothing preempted, submission order)."""
    B, kv_block, pool, reqs, script = _random_trace(300 + seed)
    B, pool = B + 2, 3 * pool                                  # room for batches: at least three slots
    chunk, tile = 256, 32
    s = sched_oracle.BatchedScheduler(B, pool, kv_block, chunk, tile)
    for p, m in reqs:
        s.add_request(p, m)
    order, decodes = [], {r: 0 for r in range(len(reqs))}
    batches = 0
    for _ in range(100000):
        waiting_before = [r.rid for r in s.waiting]
        running_before, free_before = [r.rid for r in s.running], s.free_pages
        it = s.decision()
        if it.kind == "idle":
            break
        if it.kind == "prefill":
            n = len(it.requests)
            batches += n > 1
            assert it.requests == waiting_before[:n]                               # a prefix of the queue: nobody overtakes
            assert len(running_before) + n <= B
            assert sum(-(-sum(reqs[r]) // kv_block) for r in it.requests) <= free_before
            rows = 0
            for r in it.requests:
                rows = -(-rows // tile) * tile + reqs[r][0]
            assert -(-rows // chunk) == -(-reqs[it.requests[0]][0] // chunk)       # no chunk more than the head alone takes
            assert it.tokens == sum(reqs[r][0] for r in it.requests)
            order += it.requests
        else:
            assert it.requests == running_before
            for r in it.requests:
                decodes[r] += 1
    assert order == list(range(len(reqs))) and batches > 0
    assert all(1 + decodes[r] == reqs[r][1] for r in range(len(reqs)))
    assert s.free_pages == pool and not s.running and not s.waiting


class _BatchingStandIn(_StandInEngine):
    """The stand-in engine with a batched prefill call (records one call for the whole batch)."""

    def __init__(self, B, pool, kv_block):
        super().__init__(B, pool, kv_block)
        self.batch_fn = self.corun.PREFILL_BATCH_FN(self._prefill_batch)

    def _prefill_batch(self, ctx, n, slots, tokens, lens, reserves, samplings, seeds, firsts):
        need = sum(-(-reserves[i] // self.kv_block) for i in range(n))
        if need > self.free or any(slots[i] in self.pages for i in range(n)):
            return self.corun.ENOSPACE
        off = 0
        for i in range(n):
            self.pages[slots[i]] = -(-reserves[i] // self.kv_block)
            self.step_of[slots[i]] = 1
            firsts[i] = int(seeds[i]) % 1000
            assert [tokens[off + j] for j in range(lens[i])] == [j % 97 for j in range(lens[i])]
            off += lens[i]
        self.free -= need
        self.calls.append(("prefill_batch", tuple(slots[i] for i in range(n)), tuple(lens[i] for i in range(n)),
                           tuple(int(seeds[i]) for i in range(n))))
        return 0


@pytest.mark.parametrize("seed", range(6))
def test_library_scheduler_takes_the_batched_oracles_decisions(seed):
    from paper_2608_14376_b200 import build, corun

    build.build()
    B, kv_block, pool, reqs, script = _random_trace(200 + seed)
    B, pool = B + 2, 3 * pool                                  # room for batches: at least three slots
    chunk, tile = 256, 32
    eng = _BatchingStandIn(B, pool, kv_block)
    sch = corun.Scheduler(ops=eng.ops, B=B, kv_block=kv_block, max_context=256)
    sch.enable_batched_prefill(eng.batch_fn, chunk, tile)
    ref = sched_oracle.BatchedScheduler(B, pool, kv_block, chunk, tile)
    nxt, n_batched = 0, 0
    try:
        with pytest.raises(corun.CorunError):
            sch.enable_batched_prefill(eng.batch_fn, 64, 48)                     # tile must divide the chunk
        for op, k in script + [("step", 10 ** 6)]:
            if op == "submit":
                for i, (p, m) in enumerate(reqs[nxt:nxt + k]):
                    sch.submit(np.arange(p) % 97, m, 0.7, 0.9, seed=5000 + nxt + i)
                    ref.add_request(p, m)
                nxt += k
                continue
            for _ in range(k):
                want = ref.decision()
                action, rid, n = sch.step()
                assert action == {"idle": corun.SCHED_IDLE, "prefill": corun.SCHED_PREFILL, "decode": corun.SCHED_DECODE}[want.kind]
                if want.kind == "prefill":
                    assert rid == want.requests[0] and n == len(want.requests)
                    if n > 1:
                        n_batched += 1
                        call = [c for c in eng.calls if c[0] == "prefill_batch"][-1]
                        assert call[2] == tuple(reqs[r][0] for r in want.requests)
                        assert call[3] == tuple(5000 + r for r in want.requests)
                elif want.kind == "decode":
                    assert n == len(want.requests)
                assert sch.counts() == (len(ref.waiting), len(ref.running))
                assert eng.free == ref.free_pages
                if want.kind == "idle" and nxt == len(reqs):
                    break
        assert n_batched > 0
        for rid, (p, m) in enumerate(reqs):
            toks, fin = sch.poll(rid)
            assert fin and list(toks) == [(5000 + rid) % 1000 + t for t in range(m)]
        assert eng.free == pool and not eng.pages
    finally:
        sch.close()
