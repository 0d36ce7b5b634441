"""The engine with Mixture-of-Experts feed-forward layers (tiny attention shape; 8 routed experts of 128,
top-2, one shared expert; and a renormalised top-4 of 16 without shared expert): prefill and teacher-forced
decode steps against the C oracle, bitwise invariance to slot, co-tenants and repeats, batched prefill."""
import numpy as np
import pytest

from paper_2608_14376_b200 import synth

pytestmark = pytest.mark.gpu

B, MAX_CTX = 8, 192
TOL = 3e-2


def _setup(orc, E, K, F, S, renorm, seed):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    sh = synth.TINY
    w_np = synth.make_weights_numpy(sh, seed=seed)
    m_np = synth.make_moe_numpy(sh, E, K, F, S, renorm, seed=seed)
    model = orc.Model(orc.Shape(**sh.dict()), w_np, moe=m_np)
    w_t = synth.weights_numpy_to_torch(w_np, "cuda")
    m_t = synth.moe_numpy_to_torch(m_np, "cuda")
    eng = corun.Engine(sh, w_t, B, MAX_CTX, moe=m_t)
    return sh, model, eng


@pytest.mark.parametrize("E,K,F,S,renorm", [(8, 2, 128, 1, False), (16, 4, 64, 0, True)])
def test_moe_engine_parity_and_invariance(orc, E, K, F, S, renorm):
    sh, model, eng = _setup(orc, E, K, F, S, renorm, seed=3)
    try:
        lens = [21, 150, 64, 9]
        prompts = synth.make_prompts(sh.vocab, lens, seed=31)
        slots = [5, 0, 2, 7]
        reqs = [orc.Request(model, p, 1, max_T=MAX_CTX) for p in prompts]
        worst = 0.0
        for s, p, r in zip(slots, prompts, reqs):
            r.prefill()
            eng.prefill(s, p, len(p) + 8)
            worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
        active = np.zeros(B, np.uint8); active[slots] = 1
        seeds = np.zeros(B, np.uint64)
        trace = []
        for _ in range(4):                              # teacher-forced with the oracle's greedy tokens
            for s, r in zip(slots, reqs):
                eng.force_token(s, int(np.argmax(r.logits)))
            toks = [int(np.argmax(r.logits)) for r in reqs]
            eng.decode_step(active, seeds)
            for s, r, t in zip(slots, reqs, toks):
                r.decode(force_token=t)
                worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
            trace.append([eng.logits(s).tobytes() for s in slots])
        assert worst <= TOL, worst
        assert eng.decode_launches() == 7 + 11 * sh.n_layers

        # the same requests in other slots, two of them alone, then all in one batched prefill: same bytes
        for s in slots:
            eng.release(s)
        slots2 = [1, 6, 3, 4]
        first = eng.prefill_batch(slots2, prompts, [len(p) + 8 for p in prompts])
        assert all(0 <= int(t) < sh.vocab for t in first)
        cur = [orc.Request(model, p, 1, max_T=MAX_CTX) for p in prompts]
        for r in cur:
            r.prefill()
        active = np.zeros(B, np.uint8); active[slots2] = 1
        for step in range(4):
            for s, r in zip(slots2, cur):
                eng.force_token(s, int(np.argmax(r.logits)))
            toks = [int(np.argmax(r.logits)) for r in cur]
            eng.decode_step(active, seeds)
            for r, t in zip(cur, toks):
                r.decode(force_token=t)
            assert [eng.logits(s).tobytes() for s in slots2] == trace[step]
        # one request alone (the others released): still the same bytes as among co-tenants
        for s in slots2[1:]:
            eng.release(s)
        eng.release(slots2[0])
        eng.prefill(2, prompts[0], lens[0] + 8)
        solo = orc.Request(model, prompts[0], 1, max_T=MAX_CTX)
        solo.prefill()
        active = np.zeros(B, np.uint8); active[2] = 1
        for step in range(4):
            t = int(np.argmax(solo.logits))
            eng.force_token(2, t)
            eng.decode_step(active, seeds)
            solo.decode(force_token=t)
            assert eng.logits(2).tobytes() == trace[step][0]
    finally:
        eng.close()


def test_moe_engine_served_together_equals_served_alone(orc):
    """The paper's validation protocol on the MoE decoder: requests served together (sampled, through the host
    scheduler with a pool too small for all of them) produce, bit for bit, the tokens of each served alone."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    sh = synth.TINY
    w_np = synth.make_weights_numpy(sh, seed=5)
    m_np = synth.make_moe_numpy(sh, 8, 2, 128, 1, False, seed=5)
    eng = corun.Engine(sh, synth.weights_numpy_to_torch(w_np, "cuda"), B, 128, kv_pool_blocks=24,
                       moe=synth.moe_numpy_to_torch(m_np, "cuda"))
    try:
        rng = np.random.default_rng(2)
        lens = synth.uniform_lengths(8, 70, 14, seed=8)
        prompts = synth.make_prompts(sh.vocab, lens, seed=9)
        reqs = [dict(prompt=p, max_new=int(rng.integers(2, 12)), seed=synth.request_seed(50 + i)) for i, p in enumerate(prompts)]

        def serve(subset, batched=False):
            sch = corun.Scheduler(engine=eng)
            if batched:
                sch.enable_batched_prefill()
            ids = [sch.submit(r["prompt"], r["max_new"], 0.8, 0.9, r["seed"]) for r in subset]
            shared = 0
            while True:
                action, _, n = sch.step()
                shared += action == corun.SCHED_DECODE and n >= 3
                if action == corun.SCHED_IDLE:
                    break
            out = [sch.poll(i)[0] for i in ids]
            sch.close()
            return out, shared

        together, shared = serve(reqs)
        assert shared > 0 and eng.free_blocks() == 24
        batched, _ = serve(reqs, batched=True)
        for r, a, b in zip(reqs, together, batched):
            alone, _ = serve([r])
            assert len(a) == r["max_new"]
            np.testing.assert_array_equal(alone[0], a)
            np.testing.assert_array_equal(b, a)
    finally:
        eng.close()
