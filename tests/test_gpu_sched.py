"""The host scheduler on a real engine (tiny configuration, B = 8, a KV pool too small for all
requests at once): every request's token sequence must equal, bit for bit, what the same request
produces when it is served alone on the same engine (the paper's validation of its determinism
contract), the decisions must be those of the scheduling oracle, and the first request's greedy
tokens must be the argmax of the oracle model's logits."""
import numpy as np
import pytest

from oracle import sched_oracle
from paper_2608_14376_b200 import synth
from tests.helpers import Tiny, top2_gap

pytestmark = pytest.mark.gpu

B, MAX_CTX, POOL = 8, 128, 20


@pytest.fixture(scope="module")
def tiny(orc):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return Tiny(orc)


def _requests(n=24):
    rng = np.random.default_rng(11)
    lens = synth.uniform_lengths(16, 64, n, seed=4)
    prompts = synth.make_prompts(synth.TINY.vocab, lens, seed=5)
    out = []
    for i, p in enumerate(prompts):
        greedy = i % 5 == 0
        out.append(dict(prompt=p, max_new=int(rng.integers(1, 14)), T=0.0 if greedy else 0.7, P=1.0 if greedy else 0.95,
                        seed=synth.request_seed(i)))
    return out


def _serve(sch, reqs, bursts):
    """Submits the requests in bursts between scheduling decisions; returns tokens and the decisions."""
    ids, log, nxt = [], [], 0
    for k, steps in bursts + [(0, 10 ** 6)]:
        for r in reqs[nxt:nxt + k]:
            ids.append(sch.submit(r["prompt"], r["max_new"], r["T"], r["P"], r["seed"]))
        nxt += k
        for _ in range(steps):
            action, rid, n = sch.step()
            log.append((action, rid, n))
            if action == 0 and nxt == len(reqs):
                break
    return [sch.poll(i) for i in ids], log


def test_served_together_equals_served_alone_and_follows_the_oracle(orc, tiny):
    from paper_2608_14376_b200 import corun

    reqs = _requests()
    eng = corun.Engine(tiny.sh, tiny.w_t, B, MAX_CTX, kv_pool_blocks=POOL)
    try:
        # ---- all together, arriving in bursts
        rng = np.random.default_rng(3)
        bursts, left = [], len(reqs)
        while left:
            k = int(min(left, rng.integers(1, 7)))
            bursts.append((k, int(rng.integers(0, 6))))
            left -= k
        sch = corun.Scheduler(engine=eng)
        together, log = _serve(sch, reqs, bursts)
        sch.close()
        assert all(fin and len(t) == r["max_new"] for (t, fin), r in zip(together, reqs))
        assert eng.free_blocks() == POOL
        assert any(a == corun.SCHED_DECODE and n >= 3 for a, _, n in log)        # requests did share decode iterations

        # ---- the oracle takes the same decisions
        ref = sched_oracle.Scheduler(B, POOL, 16, chunk=256)
        nxt, i = 0, 0
        for k, steps in bursts + [(0, 10 ** 6)]:
            for r in reqs[nxt:nxt + k]:
                ref.add_request(len(r["prompt"]), r["max_new"])
            nxt += k
            for _ in range(steps):
                want = ref.decision()
                action, rid, n = log[i]; i += 1
                assert action == {"idle": 0, "prefill": 1, "decode": 2}[want.kind]
                assert n == len(want.requests) and (want.kind != "prefill" or rid == want.requests[0])
                if want.kind == "idle" and nxt == len(reqs):
                    break
        assert i == len(log)

        # ---- one at a time on the same engine: identical tokens
        for r, (toks, _) in zip(reqs, together):
            sch = corun.Scheduler(engine=eng)
            alone, _ = _serve(sch, [r], [(1, 0)])
            sch.close()
            np.testing.assert_array_equal(alone[0][0], toks)

        # ---- and they are the oracle model's greedy tokens for the first request (teacher-forced with
        # the served tokens; compared wherever the oracle's top-2 gap is clear of the tolerance)
        r, served = reqs[0], list(together[0][0])
        cache = tiny.oracle.new_cache(MAX_CTX)
        lg = tiny.oracle.forward(r["prompt"], 0, cache)
        checked = 0
        for t in range(r["max_new"]):
            if top2_gap(lg) > 0.1:
                assert int(np.argmax(lg)) == served[t]
                checked += 1
            if t + 1 < r["max_new"]:
                lg = tiny.oracle.forward([served[t]], len(r["prompt"]) + t, cache)
        assert checked >= 1
    finally:
        eng.close()


def test_batched_prefill_policy_serves_the_same_tokens_and_follows_its_oracle(tiny):
    """The scheduler with batched prefill on (requests behind the head ride in the padding of its chunks):
    every request's tokens equal those under the isolated policy, bit for bit, the decisions are those of
    the batched oracle, and some prefill decision did take several requests."""
    from paper_2608_14376_b200 import corun

    reqs = _requests()
    eng = corun.Engine(tiny.sh, tiny.w_t, B, MAX_CTX, kv_pool_blocks=POOL)
    try:
        bursts = [(6, 2), (5, 3), (7, 1), (6, 4)]
        sch = corun.Scheduler(engine=eng)
        isolated, _ = _serve(sch, reqs, bursts)
        sch.close()
        sch = corun.Scheduler(engine=eng)
        sch.enable_batched_prefill()
        batched, log = _serve(sch, reqs, bursts)
        sch.close()
        assert eng.free_blocks() == POOL
        for (a, fa), (b, fb) in zip(isolated, batched):
            assert fa and fb
            np.testing.assert_array_equal(a, b)
        assert any(a == corun.SCHED_PREFILL and n > 1 for a, _, n in log)
        chunk, tile = 256, 128 // (tiny.sh.n_q_heads // tiny.sh.n_kv_heads)
        ref = sched_oracle.BatchedScheduler(B, POOL, 16, chunk, tile)
        nxt, i = 0, 0
        for k, steps in bursts + [(0, 10 ** 6)]:
            for r in reqs[nxt:nxt + k]:
                ref.add_request(len(r["prompt"]), r["max_new"])
            nxt += k
            for _ in range(steps):
                want = ref.decision()
                action, rid, n = log[i]; i += 1
                assert action == {"idle": 0, "prefill": 1, "decode": 2}[want.kind]
                assert n == len(want.requests) and (want.kind != "prefill" or rid == want.requests[0])
                if want.kind == "idle" and nxt == len(reqs):
                    break
        assert i == len(log)
    finally:
        eng.close()
