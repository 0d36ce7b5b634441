"""The engine with multi-head latent attention layers (a dense first layer, expert layers behind it): prefill and
teacher-forced decode steps against the C oracle, bitwise invariance to slot, co-tenants and batched prefill, and
the DeepSeek-V2-Lite layer shape at full width."""
import os

import numpy as np
import pytest

from paper_2608_14376_b200 import synth

pytestmark = pytest.mark.gpu

B, MAX_CTX = 8, 320
TOL = 3e-2
SMALL = synth.ModelShape(3, 256, 4, 4, 128, 384, 2048, 1e-6, 10000.0)
SMALL_MLA = dict(kv_lora_rank=256, qk_nope=128, qk_rope=32, v_head=128, first_dense=1)
SMALL_MOE = dict(n_experts=8, top_k=2, expert_ffn=128, n_shared=1, renormalize=False)


def _torch():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch


def _setup(orc, sh, mla, moe, seed, B=B, max_ctx=MAX_CTX, **kw):
    _torch()
    from paper_2608_14376_b200 import corun

    w_np, m_np = synth.make_mla_weights_numpy(sh, mla, seed=seed)
    e_np = synth.make_moe_numpy(sh, seed=seed, **moe) if moe else None
    model = orc.Model(orc.Shape(**sh.dict()), w_np, moe=e_np, mla=m_np)
    w_t, m_t = synth.mla_numpy_to_torch(w_np, m_np, "cuda")
    e_t = synth.moe_numpy_to_torch(e_np, "cuda") if moe else None
    eng = corun.Engine(sh, w_t, B, max_ctx, moe=e_t, mla=m_t, **kw)
    return model, eng


# kv_block 64: the 16-token pages of a slot in aligned runs of four, fetched by the attention kernel one run per TMA box
@pytest.mark.parametrize("first_dense,moe,kv_block", [(1, SMALL_MOE, 16), (3, None, 16), (1, SMALL_MOE, 64)])
def test_mla_engine_parity_and_invariance(orc, first_dense, moe, kv_block):
    sh = SMALL
    mla = dict(SMALL_MLA, first_dense=first_dense)
    model, eng = _setup(orc, sh, mla, moe, seed=3, kv_block=kv_block)
    try:
        lens = [21, 270, 64, 9]                          # one prompt beyond a 256-token attention split and a prefill chunk
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
            toks = [int(np.argmax(r.logits)) for r in reqs]
            for s, t in zip(slots, toks):
                eng.force_token(s, t)
            eng.decode_step(active, seeds)
            for s, r, t in zip(slots, reqs, toks):
                r.decode(force_token=t)
                worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
            trace.append([eng.logits(s).tobytes() for s in slots])
        assert worst <= TOL, worst
        # per layer: 10 around the attention (2 norms, 4 GEMMs, cache append, attention splits and combine, value split)
        # + 3 (dense feed-forward) or 4 (router, 2 GEMMs, masked SwiGLU: a kernel of its own up to 64 rows)
        n_dense = first_dense if moe else sh.n_layers
        assert eng.decode_launches() == 6 + 13 * n_dense + 14 * (sh.n_layers - n_dense) - (0 if moe else n_dense)

        # the same requests in other slots, prefilled together in shared chunks: same bytes
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
            toks = [int(np.argmax(r.logits)) for r in cur]
            for s, t in zip(slots2, toks):
                eng.force_token(s, t)
            eng.decode_step(active, seeds)
            for r, t in zip(cur, toks):
                r.decode(force_token=t)
            assert [eng.logits(s).tobytes() for s in slots2] == trace[step]
        # one request alone: still the same bytes as among co-tenants
        for s in slots2:
            eng.release(s)
        eng.prefill(2, prompts[1], lens[1] + 8)
        solo = orc.Request(model, prompts[1], 1, max_T=MAX_CTX)
        solo.prefill()
        active = np.zeros(B, np.uint8); active[2] = 1
        for step in range(4):
            t = int(np.argmax(solo.logits))
            eng.force_token(2, t)
            eng.decode_step(active, seeds)
            solo.decode(force_token=t)
            assert eng.logits(2).tobytes() == trace[step][1]
    finally:
        eng.close()


def test_mla_engine_with_more_than_64_slots(orc):
    """The decode program above 64 padded rows: the grouped up-projections then run on two blocks of rows per head and
    the expert layers in their grouped form (an expert's rows gathered into blocks of 64, routing weight and SwiGLU in
    the per-group gate / up GEMM's epilogue).  Parity with the oracle and the same bytes in other slots (rows of both
    blocks)."""
    sh, Bw = SMALL, 80
    model, eng = _setup(orc, sh, dict(SMALL_MLA), SMALL_MOE, seed=6, B=Bw, max_ctx=128)
    try:
        assert eng.decode_launches() == 6 + 13 + (13 if os.environ.get("CORUN_MOE_DECODE_DENSE") else 16) * (sh.n_layers - 1)
        prompts = synth.make_prompts(sh.vocab, [30, 77, 12, 50], seed=6)
        seeds = np.zeros(Bw, np.uint64)
        traces = []
        for slots in ([3, 70, 79, 64], [65, 0, 41, 63]):
            reqs = [orc.Request(model, p, 1, max_T=128) for p in prompts]
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


def test_mla_engine_served_together_equals_served_alone(orc):
    """The paper's validation protocol on the MLA decoder: requests served together (sampled, through the host
    scheduler with a pool too small for all of them, isolated and batched prefill) produce, bit for bit, the tokens
    of each served alone."""
    _torch()
    from paper_2608_14376_b200 import corun

    sh, mla = SMALL, dict(SMALL_MLA)
    w_np, m_np = synth.make_mla_weights_numpy(sh, mla, seed=5)
    e_np = synth.make_moe_numpy(sh, seed=5, **SMALL_MOE)
    w_t, m_t = synth.mla_numpy_to_torch(w_np, m_np, "cuda")
    eng = corun.Engine(sh, w_t, B, 128, kv_pool_blocks=24, moe=synth.moe_numpy_to_torch(e_np, "cuda"), mla=m_t)
    try:
        rng = np.random.default_rng(2)
        lens = synth.uniform_lengths(8, 70, 12, seed=8)
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


def test_mla_engine_cache_rows_are_the_oracles(orc):
    """What prefill and decode append to the latent cache (normalised latent, rotated rotary key) against the oracle's
    cache, through the debug read."""
    sh, mla = SMALL, dict(SMALL_MLA, first_dense=3)
    model, eng = _setup(orc, sh, mla, None, seed=9)
    try:
        p = synth.make_prompts(sh.vocab, [37], seed=2)[0]
        r = orc.Request(model, p, 1, max_T=MAX_CTX)
        r.prefill()
        eng.prefill(3, p, 48)
        for layer in range(sh.n_layers):
            got, _ = eng.kv_read(3, layer, 0, 37)
            ref = r.cache[0][layer, :37]
            assert got.shape == ref.shape
            assert np.abs(got - ref).max() <= 2e-2, (layer, np.abs(got - ref).max())
    finally:
        eng.close()


def test_mla_engine_at_the_deepseek_v2_lite_layer_shape(orc):
    """Full layer width (hidden 2048, 16 heads, latent 512, rope 64, dense feed-forward 10944, 64 routed experts of
    1408 top-6 + 2 shared), two layers, a small vocabulary; prompts of a few dozen tokens (the oracle's definition
    form decompresses every cached token for every query)."""
    full = synth.DEEPSEEK_V2_LITE
    sh = synth.ModelShape(2, full.hidden, full.n_q_heads, full.n_q_heads, 128, full.ffn, 4096, full.rms_eps, full.rope_theta)
    model, eng = _setup(orc, sh, dict(synth.DEEPSEEK_V2_LITE_MLA), dict(synth.DEEPSEEK_V2_LITE_MOE), seed=0, B=8, max_ctx=128)
    try:
        lens = [33, 5, 48]
        prompts = synth.make_prompts(sh.vocab, lens, seed=12)
        slots = [6, 1, 3]
        reqs = [orc.Request(model, p, 1, max_T=128) for p in prompts]
        worst = 0.0
        for s, p, r in zip(slots, prompts, reqs):
            r.prefill()
            eng.prefill(s, p, len(p) + 4)
            worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
        active = np.zeros(8, np.uint8); active[slots] = 1
        seeds = np.zeros(8, np.uint64)
        for _ in range(2):
            toks = [int(np.argmax(r.logits)) for r in reqs]
            for s, t in zip(slots, toks):
                eng.force_token(s, t)
            eng.decode_step(active, seeds)
            for s, r, t in zip(slots, reqs, toks):
                r.decode(force_token=t)
                worst = max(worst, float(np.abs(eng.logits(s) - r.logits).max()))
        assert worst <= TOL, worst
    finally:
        eng.close()


def test_mla_engine_argument_errors(orc):
    torch = _torch()
    from paper_2608_14376_b200 import corun

    sh = SMALL
    w_np, m_np = synth.make_mla_weights_numpy(sh, dict(SMALL_MLA, first_dense=3), seed=1)
    w_t, m_t = synth.mla_numpy_to_torch(w_np, m_np, "cuda")
    for bad in (dict(kv_lora_rank=128), dict(qk_nope=96), dict(qk_rope=20), dict(v_head=64), dict(first_dense=1)):
        with pytest.raises(corun.CorunError):        # first_dense below the layer count needs expert layers
            corun.Engine(sh, w_t, 4, 64, mla=dict(m_t, **bad))


def test_mla_cache_blocks_of_64_tokens_are_accounted_in_blocks(orc):
    """kv_block = 64: the pool is sized, handed out and counted in blocks of 64 tokens (four 16-token pages in a row);
    the cache rows read back are the oracle's wherever the block boundaries fall."""
    sh = SMALL
    model, eng = _setup(orc, sh, dict(SMALL_MLA), SMALL_MOE, seed=8, B=8, max_ctx=256, kv_block=64, kv_pool_blocks=10)
    try:
        assert eng.free_blocks() == 10
        prompts = synth.make_prompts(sh.vocab, [70, 9, 130], seed=12)
        eng.prefill(1, prompts[0], 78)                      # 78 tokens reserved: two blocks
        assert eng.free_blocks() == 8
        eng.prefill(5, prompts[1], 64)                      # exactly one block
        assert eng.free_blocks() == 7
        eng.prefill(2, prompts[2], 200)                     # four blocks
        assert eng.free_blocks() == 3
        with pytest.raises(Exception):
            eng.prefill(3, prompts[0], 64 * 4)              # four more do not fit
        assert eng.free_blocks() == 3
        r = orc.Request(model, prompts[2], 1, max_T=256)
        r.prefill()
        got = eng.kv_read(2, 1, 0, 130)[0]                  # layer 1, positions 0..129: across three blocks of 64
        ref = r.cache[0][1, :130]
        assert got.shape == ref.shape and float(np.abs(got - ref).max()) <= 2e-2
        eng.release(2)
        assert eng.free_blocks() == 7
        eng.release(1); eng.release(5)
        assert eng.free_blocks() == 10
    finally:
        eng.close()


@pytest.mark.parametrize("kv_block", [16, 64])
def test_mla_engine_full_house_changes_no_byte(orc, kv_block):
    """Three requests alone and among co-tenants in nearly every other slot of an 80-slot engine (rows in both blocks
    of the 65..128-row GEMMs, two row blocks per head in the grouped up-projections, expert groups of more than one
    block): the same bytes, and the oracle's values; with 16-token pages and with blocks of 64 tokens."""
    sh, Bw = SMALL, 80
    model, eng = _setup(orc, sh, dict(SMALL_MLA), SMALL_MOE, seed=6, B=Bw, max_ctx=128, kv_block=kv_block)
    try:
        prompts = synth.make_prompts(sh.vocab, [30, 77, 12], seed=6)
        tested = [41, 5, 77]
        others = [s for s in range(Bw) if s not in tested][: Bw - 8]
        fill = synth.make_prompts(sh.vocab, [9 + (i * 7) % 40 for i in range(len(others))], seed=78)
        seeds = np.zeros(Bw, np.uint64)
        traces = []
        for crowd in (False, True):
            reqs = [orc.Request(model, p, 1, max_T=128) for p in prompts]
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
