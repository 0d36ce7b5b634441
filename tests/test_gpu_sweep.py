"""Occupancy sweep at the Qwen3-8B layer shape (hidden 4096, 32 q / 8 kv heads, head_dim 128, FFN 12288):
fixed padded batch B in {1, 8, 32, 128, 256} x active fraction in {1/8, 1/2, 1}, contexts uniform in
256..8192.  Every tested request runs alone and then in three random slot permutations among random
co-tenants; its logit bytes must never change, and they must match the oracle's decode step on the
same synthetic cache rows.  The model is two layers deep with a 4096-token vocabulary so that one
engine per B fits the test budget; every GEMM keeps the full layer dimensions, so the kernels run the
same row-count paths (16, 32, 128 and 256 padded rows) as the full model would."""
import numpy as np
import pytest

from paper_2608_14376_b200 import synth
from tests.helpers import oracle_model, top2_gap

pytestmark = pytest.mark.gpu

SHAPE = synth.ModelShape(2, 4096, 32, 8, 128, 12288, 4096, 1e-6, 1e6)
MAX_CTX = 8192 + 64
TOL, GAP = 3e-2, 0.1
T, P = 0.7, 0.95


@pytest.fixture(scope="module")
def sweep_model(orc):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    if torch.cuda.get_device_properties(0).total_memory < 60e9:
        pytest.skip("needs a large-memory GPU")
    w_t = synth.make_weights_torch(SHAPE, seed=0, device="cuda")
    model = oracle_model(orc, SHAPE, synth.weights_torch_to_numpy(w_t))
    return w_t, model


def _adopt_with_cache(eng, slot, req):
    n_ctx = req["ctx"]
    eng.adopt(slot, 0, n_ctx + 2, pending=req["pending"], temperature=T, top_p=P, step=1)
    for layer in range(SHAPE.n_layers):
        eng.kv_write(slot, layer, 0, req["k"][layer], req["v"][layer])


@pytest.mark.parametrize("B", [1, 8, 32, 128, 256])
def test_sweep_invariance_and_parity(orc, sweep_model, B):
    from paper_2608_14376_b200 import corun

    w_t, model = sweep_model
    rng = np.random.default_rng(300 + B)
    n_req = min(B, 3)
    ctxs = synth.uniform_lengths(256, 8192, n_req, seed=3 + B)
    reqs = []
    for i, n_ctx in enumerate(int(c) for c in ctxs):
        k, v = [], []
        cache = model.new_cache(n_ctx + 2)
        for layer in range(SHAPE.n_layers):
            kk, vv = synth.synthetic_kv(n_ctx, SHAPE.kv_dim, 1.28, seed=(B * 10 + i) * 100 + layer)
            cache[0][layer, :n_ctx] = kk
            cache[1][layer, :n_ctx] = vv
            k.append(kk); v.append(vv)
        reqs.append(dict(ctx=n_ctx, k=k, v=v, cache=cache, pending=17 + 101 * i, seed=synth.request_seed(i)))

    eng = corun.Engine(SHAPE, w_t, B, MAX_CTX)
    try:
        # ---- each request alone (in slot 0): reference bytes, parity with the oracle, the sampled token
        worst = 0.0
        for r in reqs:
            _adopt_with_cache(eng, 0, r)
            active = np.zeros(B, np.uint8); active[0] = 1
            seeds = np.zeros(B, np.uint64); seeds[0] = r["seed"]
            toks = eng.decode_step(active, seeds)
            lg = eng.logits(0)
            ref = model.forward([r["pending"]], r["ctx"], r["cache"])
            worst = max(worst, float(np.abs(lg - ref).max()))
            if top2_gap(ref) > GAP:
                assert int(np.argmax(lg)) == int(np.argmax(ref))
            assert toks[0] == orc.sample(lg, T, P, orc.variate_u24(r["seed"], 1))[0]
            r["bytes"], r["tok"] = lg.tobytes(), int(toks[0])
            eng.release(0)
        assert worst <= TOL, worst

        # ---- among co-tenants: active fraction f, three random slot permutations each
        for f in (0.125, 0.5, 1.0):
            n_active = max(1, int(round(B * f)))
            n_tested = min(n_req, n_active)
            for _ in range(3):
                slots = rng.permutation(B)[:n_active]
                active = np.zeros(B, np.uint8)
                seeds = np.zeros(B, np.uint64)
                for i in range(n_tested):
                    _adopt_with_cache(eng, int(slots[i]), reqs[i])
                    seeds[slots[i]] = reqs[i]["seed"]
                for j, s in enumerate(slots[n_tested:]):        # co-tenants with device-generated cache rows
                    n_ctx = int(rng.integers(256, 8193))
                    eng.adopt(int(s), 0, n_ctx + 2, pending=int(rng.integers(0, SHAPE.vocab)), temperature=T, top_p=P)
                    eng.kv_fill(int(s), n_ctx, 1.28, seed=int(rng.integers(1, 1 << 30)))
                    seeds[s] = 5000 + j
                active[slots] = 1
                toks = eng.decode_step(active, seeds)
                for i in range(n_tested):
                    assert eng.logits(int(slots[i])).tobytes() == reqs[i]["bytes"], (B, f, i)
                    assert int(toks[slots[i]]) == reqs[i]["tok"]
                assert (toks[active == 0] == -1).all()
                for s in slots:
                    eng.release(int(s))
    finally:
        eng.close()
