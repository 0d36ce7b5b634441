"""Pins of the Mixture-of-Experts block oracle against things other than itself (CPU)."""
import math

import numpy as np
import pytest

from oracle import moe_oracle as mo


def _rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def test_hand_computed_routing_and_output():
    """H = 2, E = 4 experts that only scale: the router weights are chosen so that the logits are
    log 4, log 3, log 2, log 1 -> p = .4 .3 .2 .1; top-2 keeps experts 0 and 1 with .4 and .3 (no
    renormalisation).  Expert e: Wg = Wu = rows that read x0, Wd = c_e, so FFN_e(x) = c_e * silu(x0) * x0."""
    x = np.array([1.0, 0.0])
    Wr = np.array([[math.log(4), 0], [math.log(3), 0], [math.log(2), 0], [0.0, 0]])
    c = [1.0, 10.0, 100.0, 1000.0]
    Wg = np.array([[[1.0, 0.0]]] * 4)            # [E, F=1, H=2]
    Wu = np.array([[[1.0, 0.0]]] * 4)
    Wd = np.array([[[ce], [0.0]] for ce in c])   # [E, H=2, F=1]
    ids, ps, p_all = mo.router(x, Wr, 2)
    assert list(ids) == [0, 1]
    np.testing.assert_allclose(p_all, [0.4, 0.3, 0.2, 0.1], rtol=1e-12)
    Y, ids2, p2 = mo.moe_ffn(x[None], Wr, Wg, Wu, Wd, [], 2)
    s = 1.0 / (1.0 + math.exp(-1.0))             # silu(1) * 1
    np.testing.assert_allclose(Y[0], [(0.4 * 1.0 + 0.3 * 10.0) * s, 0.0], rtol=1e-12)
    # with a shared expert of weight 1 on top
    Ys, _, _ = mo.moe_ffn(x[None], Wr, Wg, Wu, Wd, [(Wg[0], Wu[0], np.array([[7.0], [0.0]]))], 2)
    np.testing.assert_allclose(Ys[0], [(0.4 + 3.0 + 7.0) * s, 0.0], rtol=1e-12)


def test_ties_go_to_the_lower_expert_id():
    x = np.array([1.0, 2.0])
    Wr = np.zeros((6, 2))                        # all logits equal
    ids, ps, _ = mo.router(x, Wr, 3)
    assert list(ids) == [0, 1, 2]
    np.testing.assert_allclose(ps, 1 / 6)
    Wr[4] = [1.0, 0.0]                           # one clear winner, the rest tied
    ids, _, _ = mo.router(x, Wr, 3)
    assert list(ids) == [4, 0, 1]


def test_all_experts_selected_and_identical_is_the_dense_ffn():
    """top_k = E with identical experts: the probabilities sum to 1, so y = FFN(x) whatever the router says."""
    H, F, E, B = 12, 20, 5, 4
    X = _rand((B, H), 1)
    wg, wu, wd = _rand((F, H), 2, 0.3), _rand((F, H), 3, 0.3), _rand((H, F), 4, 0.3)
    Wg, Wu, Wd = np.stack([wg] * E), np.stack([wu] * E), np.stack([wd] * E)
    Y, _, P = mo.moe_ffn(X, _rand((E, H), 5), Wg, Wu, Wd, [], E)
    np.testing.assert_allclose(P.sum(1), 1.0, rtol=1e-12)
    torch = pytest.importorskip("torch")
    xt = torch.tensor(X, dtype=torch.float64)
    ref = (torch.nn.functional.silu(xt @ torch.tensor(wg).T) * (xt @ torch.tensor(wu).T)) @ torch.tensor(wd).T
    np.testing.assert_allclose(Y, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_brute_force_scalar_loops_on_a_tiny_case():
    H, F, E, B, K = 5, 3, 6, 3, 2
    X, Wr = _rand((B, H), 11), _rand((E, H), 12)
    Wg, Wu, Wd = _rand((E, F, H), 13), _rand((E, F, H), 14), _rand((E, H, F), 15)
    sh = [(_rand((F, H), 16), _rand((F, H), 17), _rand((H, F), 18))]
    Y, ids, ps = mo.moe_ffn(X, Wr, Wg, Wu, Wd, sh, K)
    for b in range(B):
        logit = [sum(Wr[e][h] * X[b][h] for h in range(H)) for e in range(E)]
        den = sum(math.exp(l) for l in logit)
        p = [math.exp(l) / den for l in logit]
        chosen = sorted(range(E), key=lambda e: (-p[e], e))[:K]
        assert list(ids[b]) == chosen
        def one(wg, wu, wd, scale):
            hid = []
            for f in range(F):
                g = sum(wg[f][h] * X[b][h] for h in range(H))
                u = sum(wu[f][h] * X[b][h] for h in range(H))
                hid.append(g / (1.0 + math.exp(-g)) * u)
            return [scale * sum(wd[h][f] * hid[f] for f in range(F)) for h in range(H)]
        want = [0.0] * H
        for e in chosen:
            want = [a + c for a, c in zip(want, one(Wg[e], Wu[e], Wd[e], p[e]))]
        want = [a + c for a, c in zip(want, one(*sh[0], 1.0))]
        np.testing.assert_allclose(Y[b], want, rtol=1e-10, atol=1e-12)


def test_rows_are_independent_and_the_override_keeps_the_routers_probabilities():
    H, F, E, B, K = 8, 6, 7, 5, 3
    X, Wr = _rand((B, H), 21), _rand((E, H), 22)
    Wg, Wu, Wd = _rand((E, F, H), 23), _rand((E, F, H), 24), _rand((E, H, F), 25)
    Y, ids, ps = mo.moe_ffn(X, Wr, Wg, Wu, Wd, [], K)
    perm = np.array([3, 0, 4, 2, 1])
    Yp, idp, _ = mo.moe_ffn(X[perm], Wr, Wg, Wu, Wd, [], K)
    np.testing.assert_array_equal(Yp, Y[perm])
    np.testing.assert_array_equal(idp, ids[perm])
    # forcing the router's own choice changes nothing; forcing another choice uses that choice's probabilities
    Y2, _, _ = mo.moe_ffn(X, Wr, Wg, Wu, Wd, [], K, experts=ids)
    np.testing.assert_array_equal(Y2, Y)
    other = np.array([[0, 1, 2]] * B)
    Y3, _, p3 = mo.moe_ffn(X, Wr, Wg, Wu, Wd, [], K, experts=other)
    for b in range(B):
        _, _, p_all = mo.router(X[b], Wr, K)
        np.testing.assert_allclose(p3[b], p_all[:3])
        want = sum(p_all[e] * mo.ffn(X[b], Wg[e], Wu[e], Wd[e]) for e in range(3))
        np.testing.assert_allclose(Y3[b], want, rtol=1e-12)


def test_renormalised_gating_hand_computed():
    """The example above with renormalisation: weights .4 / .7 and .3 / .7."""
    x = np.array([1.0, 0.0])
    Wr = np.array([[math.log(4), 0], [math.log(3), 0], [math.log(2), 0], [0.0, 0]])
    Wg = np.array([[[1.0, 0.0]]] * 4)
    Wu = np.array([[[1.0, 0.0]]] * 4)
    Wd = np.array([[[ce], [0.0]] for ce in (1.0, 10.0, 100.0, 1000.0)])
    Y, ids, ps = mo.moe_ffn(x[None], Wr, Wg, Wu, Wd, [], 2, renormalize=True)
    s = 1.0 / (1.0 + math.exp(-1.0))
    np.testing.assert_allclose(ps[0], [4 / 7, 3 / 7], rtol=1e-12)
    np.testing.assert_allclose(Y[0], [(4 / 7 * 1.0 + 3 / 7 * 10.0) * s, 0.0], rtol=1e-12)
    # top_k = E renormalised is the plain softmax mixture
    Y4, _, p4 = mo.moe_ffn(x[None], Wr, Wg, Wu, Wd, [], 4, renormalize=True)
    np.testing.assert_allclose(p4[0], [0.4, 0.3, 0.2, 0.1], rtol=1e-12)


# ---- the C oracle's Mixture-of-Experts layer (used inside the full decoder) against the definition above
def _bits(a):
    from paper_2608_14376_b200 import synth
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def _vals(bits):
    from paper_2608_14376_b200 import synth
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


@pytest.mark.parametrize("renorm", [False, True])
def test_c_oracle_moe_layer_equals_the_definition(renorm):
    from oracle import oracle
    from paper_2608_14376_b200 import synth

    sh = synth.TINY
    H, E, K, F, S = sh.hidden, 6, 2, 64, 1
    rng = np.random.default_rng(5)
    NB = E + S
    Wg, Wu = _bits(rng.standard_normal((NB, F, H)) * 0.1), _bits(rng.standard_normal((NB, F, H)) * 0.1)
    Wd, Wr = _bits(rng.standard_normal((NB, H, F)) * 0.1), _bits(rng.standard_normal((E, H)) * 0.3)
    gate_up = np.concatenate([np.concatenate([Wg[e], Wu[e]], 0) for e in range(NB)], 0)
    down = np.concatenate([Wd[e] for e in range(NB)], 1)
    w = synth.make_weights_numpy(sh, seed=1)
    moe = dict(n_experts=E, top_k=K, expert_ffn=F, n_shared=S, renormalize=renorm,
               router=[Wr] * sh.n_layers, gate_up=[np.ascontiguousarray(gate_up)] * sh.n_layers,
               down=[np.ascontiguousarray(down)] * sh.n_layers)
    model = oracle.Model(oracle.Shape(**sh.dict()), w, moe=moe)
    X = rng.standard_normal((5, H)).astype(np.float32)
    shared = [(_vals(Wg[E + s]), _vals(Wu[E + s]), _vals(Wd[E + s])) for s in range(S)]
    Y, ids, ps = mo.moe_ffn(X, _vals(Wr), _vals(Wg), _vals(Wu), _vals(Wd), shared, K, renormalize=renorm)
    for b in range(5):
        y, i, p = model.moe_ffn_row(1, X[b])
        assert list(i) == list(ids[b])
        np.testing.assert_allclose(p, ps[b], rtol=1e-12)
        np.testing.assert_allclose(y, Y[b], rtol=2e-6, atol=1e-7)   # the C function returns fp32


def test_c_oracle_decoder_with_one_always_selected_expert_is_the_dense_decoder():
    """E = 1, top-1, renormalised (weight exactly 1), the expert = the dense FFN: same logits as the dense model."""
    from oracle import oracle
    from paper_2608_14376_b200 import synth

    sh = synth.TINY
    w = synth.make_weights_numpy(sh, seed=2)
    moe = dict(n_experts=1, top_k=1, expert_ffn=sh.ffn, n_shared=0, renormalize=True,
               router=[np.zeros((1, sh.hidden), np.uint16)] * sh.n_layers, gate_up=w["wgate_up"], down=w["wdown"])
    dense = oracle.Model(oracle.Shape(**sh.dict()), w)
    sparse = oracle.Model(oracle.Shape(**sh.dict()), w, moe=moe)
    toks = synth.make_prompts(sh.vocab, [9], seed=4)[0]
    a = dense.forward(toks, 0, dense.new_cache(16))
    b = sparse.forward(toks, 0, sparse.new_cache(16))
    np.testing.assert_allclose(b, a, rtol=0, atol=2e-5)
