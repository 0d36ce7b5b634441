"""GPU parity and invariance of the whole hot path on the tiny configuration:
2 layers, hidden 256, 4 query / 2 KV heads, head_dim 64, FFN 768, vocab 2048,
B = 8 with 5 active slots, prompts of 16-64 tokens, 32 greedy decode steps."""
import os

import numpy as np
import pytest

from paper_2608_14376_b200 import synth
from tests.helpers import Tiny, top2_gap

pytestmark = pytest.mark.gpu

B, MAX_CTX, STEPS = 8, 128, 32
TOL = 3e-2          # max |delta logit| against the oracle (spec tolerance)
GAP = 0.1           # greedy tokens must agree where the oracle's top-2 gap exceeds this


@pytest.fixture(scope="module")
def tiny(orc):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return Tiny(orc)


@pytest.fixture()
def engine(tiny):
    from paper_2608_14376_b200 import corun

    e = corun.Engine(tiny.sh, tiny.w_t, B, MAX_CTX)
    yield e
    e.close()


def _workload():
    slots = synth.pick_slots(B, 5, seed=7)
    lens = synth.uniform_lengths(16, 64, 5, seed=1)
    prompts = synth.make_prompts(synth.TINY.vocab, lens, seed=2)
    return slots, prompts


def test_parity_prefill_and_32_greedy_steps(orc, tiny, engine):
    slots, prompts = _workload()
    reqs, worst = {}, 0.0
    n_gap = 0
    for i, (s, p) in enumerate(zip(slots, prompts)):
        r = orc.Request(tiny.oracle, p, synth.request_seed(i), max_T=MAX_CTX)
        want = r.prefill()
        got = engine.prefill(int(s), p, len(p) + STEPS + 1, seed=synth.request_seed(i))
        lg = engine.logits(int(s))
        worst = max(worst, float(np.abs(lg - r.logits).max()))
        if top2_gap(r.logits) > GAP:
            assert got == want
            n_gap += 1
        engine.force_token(int(s), want)       # teacher forcing with the oracle's token
        reqs[int(s)] = r
    active = np.zeros(B, np.uint8); active[slots] = 1
    seeds = np.zeros(B, np.uint64)
    for i, s in enumerate(slots):
        seeds[s] = synth.request_seed(i)
    for step in range(STEPS):
        toks = engine.decode_step(active, seeds)
        for s in range(B):
            if not active[s]:
                assert toks[s] == -1
                continue
            r = reqs[s]
            want = r.decode()
            lg = engine.logits(s)
            worst = max(worst, float(np.abs(lg - r.logits).max()))
            if top2_gap(r.logits) > GAP:
                assert toks[s] == want, (step, s)
                n_gap += 1
            engine.force_token(s, want)
            assert engine.context_len(s) == r.n_ctx
    assert worst <= TOL, worst
    assert n_gap >= 10
    # the cache holds the oracle's K/V up to fp16 rounding
    s0 = int(slots[0]); r = reqs[s0]
    for layer in range(tiny.sh.n_layers):
        k, v = engine.kv_read(s0, layer, 0, r.n_ctx)
        np.testing.assert_allclose(k, r.cache[0][layer, :r.n_ctx], atol=2e-3, rtol=2e-3)
        np.testing.assert_allclose(v, r.cache[1][layer, :r.n_ctx], atol=2e-3, rtol=2e-3)


def _run_request(engine, slot, prompt, seed, cotenants, steps, temperature=0.0, top_p=1.0):
    """Prefills `prompt` into `slot` (and co-tenant prompts into other slots), decodes `steps`
    steps and returns the target's logit rows (bytes) and tokens."""
    first = engine.prefill(slot, prompt, len(prompt) + steps + 1, temperature, top_p, seed)
    rows = [engine.logits(slot).tobytes()]
    toks = [first]
    active = np.zeros(B, np.uint8); active[slot] = 1
    seeds = np.zeros(B, np.uint64); seeds[slot] = seed
    for s, (p, sd) in cotenants.items():
        engine.prefill(s, p, len(p) + steps + 1, temperature, top_p, sd)
        active[s] = 1; seeds[s] = sd
    for _ in range(steps):
        out = engine.decode_step(active, seeds)
        rows.append(engine.logits(slot).tobytes())
        toks.append(int(out[slot]))
    for s in list(cotenants) + [slot]:
        engine.release(s)
    return rows, toks


def test_logits_bitwise_invariant_to_slot_cotenants_and_repeats(tiny, engine):
    rng = np.random.default_rng(11)
    prompts = synth.make_prompts(tiny.sh.vocab, [23, 40, 17, 64, 31, 50, 19], seed=12)
    target, seed = prompts[0], 1000
    base_rows, base_toks = _run_request(engine, 0, target, seed, {}, 8)
    # alone in every slot
    for slot in range(1, B):
        rows, toks = _run_request(engine, slot, target, seed, {}, 8)
        assert rows == base_rows and toks == base_toks, slot
    # three random slot permutations with random co-tenants (different prompts, seeds, counts)
    for trial in range(3):
        perm = rng.permutation(B)
        slot = int(perm[0])
        n_co = int(rng.integers(1, B))
        co = {int(perm[1 + j]): (prompts[1 + (j + trial) % 6], 2000 + 10 * trial + j) for j in range(n_co)}
        rows, toks = _run_request(engine, slot, target, seed, co, 8)
        assert rows == base_rows and toks == base_toks, trial
    # repeated run
    rows, toks = _run_request(engine, 0, target, seed, {}, 8)
    assert rows == base_rows and toks == base_toks


def test_sampled_decoding_is_invariant_and_matches_S_on_gpu_logits(orc, tiny, engine):
    prompts = synth.make_prompts(tiny.sh.vocab, [30, 45, 20], seed=21)
    T, P, seed = 0.7, 0.95, 1042
    rows, toks = _run_request(engine, 2, prompts[0], seed, {}, 12, T, P)
    rows2, toks2 = _run_request(engine, 6, prompts[0], seed, {1: (prompts[1], 7), 2: (prompts[2], 8)}, 12, T, P)
    assert rows == rows2 and toks == toks2
    assert len(set(toks)) > 3
    checked = 0
    for t, (row, tok) in enumerate(zip(rows, toks)):
        lg = np.frombuffer(row, np.float32)
        want, _ = orc.sample(lg, T, P, orc.variate_u24(seed, t))
        assert tok == want, t
        plain, plain_margin = orc.sample_plain(lg, T, P, orc.variate_u24(seed, t))   # the plain fp64 definition
        assert plain_margin < 1e-6 or tok == plain, t
        checked += 1
    assert checked == 13
    # a different seed draws different variates
    _, toks3 = _run_request(engine, 2, prompts[0], seed + 1, {}, 12, T, P)
    assert toks3 != toks


def test_eager_launches_equal_graph_replay(tiny, engine):
    prompt = synth.make_prompts(tiny.sh.vocab, [33], seed=31)[0]
    rows_g, toks_g = _run_request(engine, 3, prompt, 5, {}, 6)
    engine.set_eager(True)
    rows_e, toks_e = _run_request(engine, 3, prompt, 5, {}, 6)
    engine.set_eager(False)
    assert rows_g == rows_e and toks_g == toks_e
    assert engine.decode_launches() == 7 + 9 * tiny.sh.n_layers


def test_padding_rows_change_nothing_and_report_minus_one(tiny, engine):
    prompt = synth.make_prompts(tiny.sh.vocab, [20], seed=41)[0]
    engine.prefill(1, prompt, 40)
    engine.prefill(4, prompt, 40)
    active = np.zeros(B, np.uint8); active[1] = 1          # slot 4 occupied but not active
    out = engine.decode_step(active, np.zeros(B, np.uint64))
    assert out[1] >= 0 and all(out[s] == -1 for s in range(B) if s != 1)
    assert engine.context_len(1) == 21 and engine.context_len(4) == 20
    k0, _ = engine.kv_read(4, 0, 0, 20)
    out = engine.decode_step(active, np.zeros(B, np.uint64))
    k1, _ = engine.kv_read(4, 0, 0, 20)
    np.testing.assert_array_equal(k0, k1)


def test_a_slots_logits_follow_the_slot_whatever_row_it_takes(tiny, engine):
    """The rows of a decode step are the slots with a request first, so a slot's row changes with its co-tenants:
    the logits of a slot are its prefill's until it decodes (other slots' steps in between do not touch them), then
    those of its own row of the last step it took part in."""
    prompts = synth.make_prompts(tiny.sh.vocab, [20, 33, 27], seed=43)
    engine.prefill(6, prompts[0], 60)
    after_prefill = engine.logits(6).tobytes()
    engine.prefill(2, prompts[1], 60)
    engine.prefill(0, prompts[2], 60)
    seeds = np.zeros(B, np.uint64)
    only = np.zeros(B, np.uint8); only[[0, 2]] = 1          # slot 6 occupied, not active: rows 0 and 1 are slots 0 and 2
    engine.decode_step(only, seeds)
    engine.decode_step(only, seeds)
    assert engine.logits(6).tobytes() == after_prefill
    a = np.zeros(B, np.uint8); a[6] = 1                       # alone: slot 6 is row 0
    engine.decode_step(a, seeds)
    alone = engine.logits(6).tobytes()
    assert alone != after_prefill
    # the same step of the same request behind two co-tenants (row 2), on a fresh engine state
    engine.release(6); engine.release(2); engine.release(0)
    engine.prefill(6, prompts[0], 60)
    engine.prefill(2, prompts[1], 60)
    engine.prefill(0, prompts[2], 60)
    both = np.zeros(B, np.uint8); both[[0, 2, 6]] = 1
    out = engine.decode_step(both, seeds)
    assert engine.logits(6).tobytes() == alone
    assert all(out[s] >= 0 for s in (0, 2, 6)) and all(out[s] == -1 for s in range(B) if s not in (0, 2, 6))


def test_error_paths(tiny, engine):
    from paper_2608_14376_b200 import corun

    prompt = synth.make_prompts(tiny.sh.vocab, [16], seed=51)[0]

    def status(fn):
        with pytest.raises(corun.CorunError) as ei:
            fn()
        return ei.value.status

    assert status(lambda: engine.prefill(B, prompt, 32)) == corun.ESLOT
    assert status(lambda: engine.prefill(0, prompt, MAX_CTX + 1)) == corun.EINVAL
    assert status(lambda: engine.prefill(0, prompt, 8)) == corun.EINVAL          # reserve < prompt
    assert status(lambda: engine.prefill(0, [tiny.sh.vocab], 8)) == corun.EINVAL
    assert status(lambda: engine.release(0)) == corun.ESLOT
    engine.prefill(0, prompt, 17)
    assert status(lambda: engine.prefill(0, prompt, 32)) == corun.ESLOT           # busy
    active = np.zeros(B, np.uint8); active[0] = 1
    engine.decode_step(active, np.zeros(B, np.uint64))                            # ctx 16 -> 17 = reserve
    assert status(lambda: engine.decode_step(active, np.zeros(B, np.uint64))) == corun.ECTX
    assert engine.context_len(0) == 17                                            # refused step changed nothing
    active[0] = 0; active[3] = 1                                                  # slot 3 is empty
    assert status(lambda: engine.decode_step(active, np.zeros(B, np.uint64))) == corun.ESLOT
    engine.release(0)


def test_admission_reserves_the_full_sequence(tiny):
    from paper_2608_14376_b200 import corun

    e = corun.Engine(tiny.sh, tiny.w_t, B, MAX_CTX, kv_pool_blocks=10)
    prompt = synth.make_prompts(tiny.sh.vocab, [16], seed=61)[0]
    assert e.free_blocks() == 10
    e.prefill(0, prompt, 100)                 # ceil(100/16) = 7 pages
    assert e.free_blocks() == 3
    with pytest.raises(corun.CorunError) as ei:
        e.prefill(1, prompt, 64)              # needs 4 > 3
    assert ei.value.status == corun.ENOSPACE
    assert e.free_blocks() == 3               # a refused admission takes nothing
    e.prefill(1, prompt, 48)
    e.release(0)
    assert e.free_blocks() == 7
    e.close()


def test_chunked_prefill_matches_oracle_and_single_chunk(orc, tiny):
    """Prompt longer than the prefill chunk: chunks are a function of the length only."""
    from paper_2608_14376_b200 import corun

    prompt = synth.make_prompts(tiny.sh.vocab, [75], seed=71)[0]
    r = orc.Request(tiny.oracle, prompt, 1, max_T=MAX_CTX)
    r.prefill()
    old = os.environ.get("CORUN_PREFILL_CHUNK")
    os.environ["CORUN_PREFILL_CHUNK"] = "32"
    try:
        e = corun.Engine(tiny.sh, tiny.w_t, B, MAX_CTX)
    finally:
        if old is None:
            del os.environ["CORUN_PREFILL_CHUNK"]
        else:
            os.environ["CORUN_PREFILL_CHUNK"] = old
    e.prefill(5, prompt, 100)
    lg = e.logits(5)
    assert np.abs(lg - r.logits).max() <= TOL
    a = lg.tobytes()
    e.release(5)
    e.prefill(2, prompt, 100)
    assert e.logits(2).tobytes() == a
    e.close()


def test_adopted_slot_with_written_cache_matches_oracle(orc, tiny, engine):
    """Synthetic-KV route used for long contexts: write K/V rows, then decode one token."""
    sh = tiny.sh
    n = 90
    cache = tiny.oracle.new_cache(MAX_CTX)
    for layer in range(sh.n_layers):
        k, v = synth.synthetic_kv(n, sh.kv_dim, 0.3, seed=100 + layer)
        cache[0][layer, :n] = k
        cache[1][layer, :n] = v
    engine.adopt(6, 0, n + 4, pending=17)
    for layer in range(sh.n_layers):
        engine.kv_write(6, layer, 0, cache[0][layer, :n], cache[1][layer, :n])
    assert engine.context_len(6) == n
    want = tiny.oracle.forward([17], n, cache)
    active = np.zeros(B, np.uint8); active[6] = 1
    engine.decode_step(active, np.zeros(B, np.uint64))
    assert np.abs(engine.logits(6) - want).max() <= TOL


@pytest.mark.parametrize("n_ctx", [255, 256, 257, 700, 1023, 8191, 8193, 9000])
def test_multi_split_attention_matches_oracle(orc, tiny, n_ctx):
    """Contexts spanning several 128-token splits and ragged tails (synthetic cache rows), up to more than
    64 splits (the combine's general path)."""
    from paper_2608_14376_b200 import corun

    sh = tiny.sh
    e = corun.Engine(sh, tiny.w_t, B, 1040 if n_ctx < 1024 else 9216)
    cache = tiny.oracle.new_cache(n_ctx + 2)
    e.adopt(2, 0, n_ctx + 2, pending=33)
    for layer in range(sh.n_layers):
        k, v = synth.synthetic_kv(n_ctx, sh.kv_dim, 0.5, seed=7 * n_ctx + layer)
        cache[0][layer, :n_ctx] = k
        cache[1][layer, :n_ctx] = v
        e.kv_write(2, layer, 0, k, v)
    want = tiny.oracle.forward([33], n_ctx, cache)
    active = np.zeros(B, np.uint8); active[2] = 1
    e.decode_step(active, np.zeros(B, np.uint64))
    err = float(np.abs(e.logits(2) - want).max())
    k_back, v_back = e.kv_read(2, 1, 0, n_ctx)
    np.testing.assert_array_equal(k_back, cache[0][1, :n_ctx])
    e.close()
    assert err <= TOL, err


@pytest.mark.parametrize("nq,nkv,hd", [(4, 4, 64), (8, 1, 64), (4, 2, 128), (8, 8, 128)])
def test_other_head_groupings_match_oracle(orc, nq, nkv, hd):
    """Query heads per KV head 1, 2 and 8 (the tiny and the Qwen shapes have 2 and 4), both head sizes:
    prefill of a prompt that spans several attention splits, then teacher-forced decode steps among
    co-tenants, against the oracle."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun
    from tests.helpers import oracle_model

    sh = synth.ModelShape(2, 256, nq, nkv, hd, 512, 1024, 1e-6, 1e4)
    w_np = synth.make_weights_numpy(sh, seed=nq * 10 + nkv)
    w_t = synth.weights_numpy_to_torch(w_np, "cuda")
    model = oracle_model(orc, sh, w_np)
    eng = corun.Engine(sh, w_t, 4, 512)
    try:
        prompts = synth.make_prompts(sh.vocab, [300, 37, 130], seed=nq + nkv)
        reqs, worst = [], 0.0
        for slot, p in zip((2, 0, 3), prompts):
            r = orc.Request(model, p, 77 + slot, max_T=512)
            want = r.prefill()
            eng.prefill(slot, p, len(p) + 8, seed=77 + slot)
            worst = max(worst, float(np.abs(eng.logits(slot) - r.logits).max()))
            eng.force_token(slot, want)
            reqs.append((slot, r))
        active = np.zeros(4, np.uint8); active[[2, 0, 3]] = 1
        seeds = np.zeros(4, np.uint64)
        for step in range(4):
            toks = eng.decode_step(active, seeds)
            assert toks[1] == -1
            for slot, r in reqs:
                want = r.decode()
                worst = max(worst, float(np.abs(eng.logits(slot) - r.logits).max()))
                if top2_gap(r.logits) > GAP:
                    assert toks[slot] == want
                eng.force_token(slot, want)
        assert worst <= TOL, worst
    finally:
        eng.close()


def test_attention_item_assignment_changes_no_bit(tiny):
    """Which SM computes which split of a request's attention has no influence on any value: the
    ablation mode, in which a CTA takes whole (row, kv head) pairs instead of single splits, yields
    the same logit bytes and tokens as the request-local split."""
    from paper_2608_14376_b200 import corun

    sh = tiny.sh
    ctxs = [700, 130, 1023, 257, 64]
    slots = [6, 1, 3, 0, 5]
    out = []
    for whole in (0, 1):
        if whole:
            os.environ["CORUN_ATTN_WHOLE_PAIRS"] = "1"
        try:
            e = corun.Engine(sh, tiny.w_t, B, 1040)
        finally:
            os.environ.pop("CORUN_ATTN_WHOLE_PAIRS", None)
        for i, (s, n) in enumerate(zip(slots, ctxs)):
            e.adopt(s, 0, n + 8, pending=11 + i, temperature=0.7, top_p=0.95)
            e.kv_fill(s, n, 0.5, seed=40 + i)
        active = np.zeros(B, np.uint8); active[slots] = 1
        seeds = np.arange(B, dtype=np.uint64) + 9
        got = []
        for _ in range(3):
            toks = e.decode_step(active, seeds)
            got.append((toks.tobytes(), b"".join(e.logits(s).tobytes() for s in slots)))
        e.close()
        out.append(got)
    assert out[0] == out[1]


def test_batched_prefill_equals_isolated_prefill(tiny):
    """Prefill requests batched with other prefill requests (the paper's future work on prefill): prompts
    that share chunks -- pieces starting on attention-tile boundaries, a prompt cut differently than when
    it runs alone -- leave the same cache, logits, first tokens and following decode steps, byte for byte,
    as isolated prefill of each."""
    from paper_2608_14376_b200 import corun

    sh = tiny.sh
    lens = [5, 70, 64, 1, 300, 33, 129]
    slots = [3, 0, 6, 1, 7, 2, 5]
    prompts = synth.make_prompts(sh.vocab, lens, seed=91)
    seeds = np.array([synth.request_seed(i) for i in range(len(lens))], np.uint64)
    res = [n + 8 for n in lens]
    T, P_ = 0.7, 0.95

    def after(e):
        active = np.zeros(B, np.uint8); active[slots] = 1
        sd = np.zeros(B, np.uint64); sd[slots] = seeds
        out = []
        out.append(b"".join(e.logits(s).tobytes() for s in slots))
        for layer in range(sh.n_layers):
            for s, n in zip(slots, lens):
                k, v = e.kv_read(s, layer, 0, n)
                out.append(k.tobytes() + v.tobytes())
        for _ in range(3):
            out.append(e.decode_step(active, sd).tobytes())
            out.append(b"".join(e.logits(s).tobytes() for s in slots))
        return out

    e = corun.Engine(sh, tiny.w_t, B, 512)
    first_iso = [e.prefill(s, p, r, T, P_, seed=int(sd)) for s, p, r, sd in zip(slots, prompts, res, seeds)]
    iso = after(e)
    for s in slots:
        e.release(s)
    first_bat = e.prefill_batch(slots, prompts, res, T, P_, seeds)
    bat = after(e)
    assert list(first_bat) == first_iso
    assert bat == iso
    # error paths: a busy slot, a slot named twice, a reservation beyond max_context -- the engine stays as it was
    with pytest.raises(corun.CorunError):
        e.prefill_batch([slots[0]], [prompts[0]], [res[0]])
    e.release(slots[0]); e.release(slots[1])
    free = e.free_blocks()
    with pytest.raises(corun.CorunError):
        e.prefill_batch([slots[0], slots[0]], prompts[:2], res[:2])
    with pytest.raises(corun.CorunError):
        e.prefill_batch([slots[0], slots[1]], prompts[:2], [res[0], 10 ** 6])
    assert e.free_blocks() == free
    e.close()
    # reservations that do not all fit: nothing is taken
    small = corun.Engine(sh, tiny.w_t, B, 512, kv_pool_blocks=12)
    with pytest.raises(corun.CorunError) as ei:
        small.prefill_batch([0, 1], prompts[1:3], [100, 100])     # 7 + 7 pages of 16 tokens
    assert ei.value.status == corun.ENOSPACE and small.free_blocks() == 12
    assert list(small.prefill_batch([0], prompts[1:2], [100], T, P_, seeds[1:2])) == [first_iso[1]]
    small.close()


@pytest.mark.parametrize("n", [129, 1100, 1793])
def test_long_prompt_prefill_matches_oracle(orc, tiny, n):
    """Prompts of 2, 9 and 15 key blocks of 128 tokens (odd and even counts for the two CTAs of a tile's
    cluster, several chunks): last-position logits and the cache against the oracle, then one decode step."""
    from paper_2608_14376_b200 import corun

    prompt = synth.make_prompts(tiny.sh.vocab, [n], seed=500 + n)[0]
    r = orc.Request(tiny.oracle, prompt, 1, max_T=n + 8)
    r.prefill()
    e = corun.Engine(tiny.sh, tiny.w_t, B, n + 8)
    e.prefill(4, prompt, n + 4)
    assert np.abs(e.logits(4) - r.logits).max() <= TOL
    for layer in range(tiny.sh.n_layers):
        k, v = e.kv_read(4, layer, 0, n)
        np.testing.assert_allclose(k, r.cache[0][layer, :n], atol=2e-3, rtol=2e-3)
        np.testing.assert_allclose(v, r.cache[1][layer, :n], atol=2e-3, rtol=2e-3)
    tok = int(np.argmax(r.logits))
    e.force_token(4, tok)
    active = np.zeros(B, np.uint8); active[4] = 1
    e.decode_step(active, np.zeros(B, np.uint64))
    r.decode(force_token=tok)
    assert np.abs(e.logits(4) - r.logits).max() <= TOL
    e.close()
