"""The engine with Mixture-of-Experts feed-forward layers (tiny attention shape; 8 routed experts of 128,
top-2, one shared expert; and a renormalised top-4 of 16 without shared expert): prefill and teacher-forced
decode steps against the C oracle, bitwise invariance to slot, co-tenants and repeats, batched prefill."""
import os

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
        assert eng.decode_launches() == 7 + 11 * sh.n_layers   # per layer: 4 GEMMs, 2 norms, RoPE, attention (splits, combine), router, masked SwiGLU

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


def test_moe_engine_with_more_than_64_slots(orc):
    """Above 64 padded rows the decode program runs the expert layers in their grouped form (an expert's rows gathered
    into blocks of 64; routing weight and SwiGLU in the epilogue of the per-group gate / up GEMM): parity with the
    oracle and the same bytes in other slots."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    sh, Bw = synth.TINY, 96
    w_np = synth.make_weights_numpy(sh, seed=4)
    m_np = synth.make_moe_numpy(sh, 8, 2, 128, 1, False, seed=4)
    model = orc.Model(orc.Shape(**sh.dict()), w_np, moe=m_np)
    eng = corun.Engine(sh, synth.weights_numpy_to_torch(w_np, "cuda"), Bw, MAX_CTX, moe=synth.moe_numpy_to_torch(m_np, "cuda"))
    try:
        # per layer: 2 norms, QKV, RoPE, attention (splits, combine), O, router, grouping, gather, 2 grouped GEMMs, combine
        # (CORUN_MOE_DECODE_DENSE=1 forces the form without groups: 10 per layer, the SwiGLU in the first GEMM's epilogue)
        assert eng.decode_launches() == 7 + (10 if os.environ.get("CORUN_MOE_DECODE_DENSE") else 13) * sh.n_layers
        prompts = synth.make_prompts(sh.vocab, [30, 77, 12], seed=6)
        seeds = np.zeros(Bw, np.uint64)
        traces = []
        for slots in ([3, 70, 95], [64, 0, 41]):
            reqs = [orc.Request(model, p, 1, max_T=MAX_CTX) for p in prompts]
            worst = 0.0
            for s, p, r in zip(slots, prompts, reqs):
                r.prefill()
                eng.prefill(s, p, len(p) + 8)
            active = np.zeros(Bw, np.uint8); active[slots] = 1
            trace = []
            for _ in range(3):
                toks = [int(np.argmax(r.logits)) for r in reqs]
                for s, t in zip(slots, toks):
                    eng.force_token(s, t)
                eng.decode_step(active, seeds)
                for s, r, t in zip(slots, reqs, toks):
                    r.decode(force_token=t)
                    worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
                trace.append([eng.logits(s).tobytes() for s in slots])
            assert worst <= TOL, worst
            traces.append(trace)
            for s in slots:
                eng.release(s)
        assert traces[0] == traces[1]
    finally:
        eng.close()


@pytest.mark.parametrize("Bw", [96, 200])
def test_moe_engine_full_house_changes_no_byte(orc, Bw):
    """The tested requests alone (three rows: one block of rows, a few small expert groups) and among co-tenants in
    nearly every other slot (rows in every block of 64 / 128 rows, expert groups of several blocks, the tested requests
    somewhere in the middle of the step's rows): the same bytes, and the oracle's values."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    sh = synth.TINY
    w_np = synth.make_weights_numpy(sh, seed=4)
    m_np = synth.make_moe_numpy(sh, 8, 2, 128, 1, False, seed=4)
    model = orc.Model(orc.Shape(**sh.dict()), w_np, moe=m_np)
    eng = corun.Engine(sh, synth.weights_numpy_to_torch(w_np, "cuda"), Bw, MAX_CTX, moe=synth.moe_numpy_to_torch(m_np, "cuda"))
    try:
        prompts = synth.make_prompts(sh.vocab, [30, 77, 12], seed=6)
        tested = [Bw // 2 + 1, 5, Bw - 3]
        others = [s for s in range(Bw) if s not in tested][: Bw - 8]
        fill = synth.make_prompts(sh.vocab, [9 + (i * 7) % 40 for i in range(len(others))], seed=77)
        seeds = np.zeros(Bw, np.uint64)
        traces = []
        for crowd in (False, True):
            reqs = [orc.Request(model, p, 1, max_T=MAX_CTX) for p in prompts]
            for s, p, r in zip(tested, prompts, reqs):
                r.prefill()
                eng.prefill(s, p, len(p) + 8)
            active = np.zeros(Bw, np.uint8); active[tested] = 1
            if crowd:
                for s, p in zip(others, fill):
                    eng.prefill(s, p, len(p) + 8)
                active[others] = 1
            worst, trace = 0.0, []
            for _ in range(3):
                toks = [int(np.argmax(r.logits)) for r in reqs]
                for s, t in zip(tested, toks):
                    eng.force_token(s, t)
                eng.decode_step(active, seeds)
                for s, r, t in zip(tested, reqs, toks):
                    r.decode(force_token=t)
                    worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
                trace.append([eng.logits(s).tobytes() for s in tested])
            assert worst <= TOL, worst
            traces.append(trace)
            for s in range(Bw):
                if active[s]:
                    eng.release(s)
        assert traces[0] == traces[1]
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


def test_moe_engine_at_the_qwen3_30b_a3b_layer_shape(orc):
    """Full layer width of the workload bench.py times for the MoE decoder (hidden 2048, 32 q / 4 kv heads of
    128, 128 experts of 768, top-8 renormalised, B = 64), two layers deep with a 4096-token vocabulary so that
    the oracle can follow: one decode step over synthetic cache rows against the oracle, then the same
    requests in other slots among other co-tenants, byte for byte."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    if torch.cuda.get_device_properties(0).total_memory < 40e9:
        pytest.skip("needs a large-memory GPU")
    from paper_2608_14376_b200 import corun

    sh = synth.ModelShape(2, 2048, 32, 4, 128, 64, 4096, 1e-6, 1e6)
    cfg = dict(synth.QWEN3_30B_A3B_MOE)
    w_t = synth.make_weights_torch(sh, seed=0, device="cuda", dense_ffn=False)
    m_t = synth.make_moe_torch(sh, seed=0, device="cuda", **cfg)
    w_np = synth.weights_torch_to_numpy({k: v for k, v in w_t.items() if k not in ("wgate_up", "wdown")})
    w_np["wgate_up"] = [np.zeros((128, sh.hidden), np.uint16)] * sh.n_layers     # unused placeholders
    w_np["wdown"] = [np.zeros((sh.hidden, 64), np.uint16)] * sh.n_layers
    m_np = dict(cfg, **{k: [t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16) for t in m_t[k]]
                        for k in ("router", "gate_up", "down")})
    model = orc.Model(orc.Shape(**sh.dict()), w_np, moe=m_np)
    Bq, max_ctx = 64, 2304
    eng = corun.Engine(sh, w_t, Bq, max_ctx, moe=m_t)
    try:
        rng = np.random.default_rng(12)
        ctxs = [2000, 700, 129]
        reqs = []
        for i, n_ctx in enumerate(ctxs):
            cache = model.new_cache(n_ctx + 2)
            kv = []
            for layer in range(sh.n_layers):
                k, v = synth.synthetic_kv(n_ctx, sh.kv_dim, 1.28, seed=900 + 10 * i + layer)
                cache[0][layer, :n_ctx], cache[1][layer, :n_ctx] = k, v
                kv.append((k, v))
            reqs.append(dict(ctx=n_ctx, kv=kv, cache=cache, pending=41 + 17 * i))

        def place(slot, r):
            eng.adopt(slot, 0, r["ctx"] + 2, pending=r["pending"], temperature=0.7, top_p=0.95, step=1)
            for layer, (k, v) in enumerate(r["kv"]):
                eng.kv_write(slot, layer, 0, k, v)

        slots = [3, 40, 63]
        for s, r in zip(slots, reqs):
            place(s, r)
        active = np.zeros(Bq, np.uint8); active[slots] = 1
        seeds = np.zeros(Bq, np.uint64)
        eng.decode_step(active, seeds)
        worst = 0.0
        for s, r in zip(slots, reqs):
            ref = model.forward([r["pending"]], r["ctx"], r["cache"])
            lg = eng.logits(s)
            worst = max(worst, float(np.abs(lg - ref).max()))
            r["bytes"] = lg.tobytes()
        assert worst <= TOL, worst
        for s in slots:
            eng.release(s)
        # other slots, 20 co-tenants with device-generated cache rows
        slots2 = [17, 0, 31]
        for s, r in zip(slots2, reqs):
            place(s, r)
        others = [s for s in rng.permutation(Bq) if s not in slots2][:20]
        for j, s in enumerate(others):
            n_ctx = int(rng.integers(64, 2000))
            eng.adopt(int(s), 0, n_ctx + 2, pending=int(rng.integers(0, sh.vocab)), temperature=0.7, top_p=0.95)
            eng.kv_fill(int(s), n_ctx, 1.28, seed=7000 + j)
        active = np.zeros(Bq, np.uint8); active[slots2] = 1; active[others] = 1
        eng.decode_step(active, seeds)
        for s, r in zip(slots2, reqs):
            assert eng.logits(s).tobytes() == r["bytes"]
    finally:
        eng.close()


def test_moe_engine_argument_errors(orc):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    sh = synth.TINY
    w_t = synth.weights_numpy_to_torch(synth.make_weights_numpy(sh, seed=1), "cuda")
    good = synth.moe_numpy_to_torch(synth.make_moe_numpy(sh, 8, 2, 128, 1), "cuda")
    for bad in (dict(top_k=0), dict(top_k=9), dict(n_experts=0), dict(expert_ffn=100), dict(n_shared=-1)):
        with pytest.raises(corun.CorunError) as ei:
            corun.Engine(sh, w_t, B, MAX_CTX, moe=dict(good, **bad))
        assert ei.value.status == corun.EINVAL
    eng = corun.Engine(sh, w_t, B, MAX_CTX, moe=good)      # and the good one still initialises
    assert eng.decode_launches() == 7 + 11 * sh.n_layers   # per layer: 4 GEMMs, 2 norms, RoPE, attention (splits, combine), router, masked SwiGLU
    eng.close()
