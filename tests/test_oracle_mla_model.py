"""Pins of the C oracle's multi-head latent attention (MLA) decoder: its attention step against the numpy
definition (oracle/mla_oracle.py, itself pinned in test_mla_oracle.py), the whole forward pass against a
composition of separately pinned pieces written here in numpy fp64 (so that a wrong offset into the fused
projection, a rotation at the wrong position, a transposed up-projection or a dropped residual shows), and
prefill against token-by-token decode on the same cache."""
import ctypes as C

import numpy as np
import pytest

from oracle import mla_oracle as ml
from oracle import moe_oracle as mo
from paper_2608_14376_b200 import synth

SH = synth.ModelShape(2, 64, 3, 3, 16, 96, 50, 1e-6, 10000.0)
MLA = dict(kv_lora_rank=24, qk_nope=16, qk_rope=8, v_head=12, first_dense=1)
MOE = dict(n_experts=4, top_k=2, expert_ffn=32, n_shared=1, renormalize=False)


def _f(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def _model(orc, seed=0, std=0.3):
    w, m = synth.make_mla_weights_numpy(SH, MLA, seed=seed, std=std)
    rng = np.random.default_rng(seed + 5)
    for l in range(SH.n_layers):                         # gains that are not all one, so that they show
        m["kv_norm"][l] = synth.f32_to_bf16_bits((1.0 + 0.2 * rng.standard_normal(MLA["kv_lora_rank"])).astype(np.float32))
        w["attn_norm"][l] = synth.f32_to_bf16_bits((1.0 + 0.2 * rng.standard_normal(SH.hidden)).astype(np.float32))
    moe = synth.make_moe_numpy(SH, seed=seed, std=std, router_std=1.0, **MOE)
    return w, m, moe, orc.Model(orc.Shape(**SH.dict()), w, moe=moe, mla=m)


def test_attention_step_is_the_numpy_definition(orc):
    rng = np.random.default_rng(1)
    nh, rank, nope, rope, vh, T = 3, 24, 16, 8, 12, 9
    wkv_b = synth.f32_to_bf16_bits((rng.standard_normal((nh * (nope + vh), rank)) * 0.4).astype(np.float32))
    q = rng.standard_normal((nh, nope + rope)).astype(np.float32)
    Cc = rng.standard_normal((T, rank + rope)).astype(np.float32)
    out = np.zeros((nh, vh), np.float32)
    for p in (0, 3, T - 1):
        orc.lib().orc_mla_attention(q.ctypes.data, Cc.ctypes.data, rank + rope, p, nh, rank, nope, rope, vh, wkv_b.ctypes.data,
                                    out.ctypes.data)
        W = _f(wkv_b).reshape(nh, nope + vh, rank)
        ref = ml.attend(q[:, :nope], q[:, nope:], Cc[:p + 1, :rank], Cc[:p + 1, rank:], W[:, :nope], W[:, nope:])
        assert np.abs(out - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())


def _rms(x, g, eps):
    return x / np.sqrt(np.mean(x * x) + eps) * g


def _rot(v, pos, theta):
    half = v.shape[0] // 2
    ang = pos * theta ** (-2.0 * np.arange(half) / v.shape[0])
    a, b = v[:half], v[half:]
    return np.concatenate([a * np.cos(ang) - b * np.sin(ang), a * np.sin(ang) + b * np.cos(ang)])


def _forward_numpy(w, m, moe, tokens):
    """All-position logits of one request, every step rounded to fp32 where the C oracle stores fp32."""
    nh, rank, nope, rope, vh = SH.n_q_heads, MLA["kv_lora_rank"], MLA["qk_nope"], MLA["qk_rope"], MLA["v_head"]
    f32 = lambda a: np.asarray(a, np.float64).astype(np.float32).astype(np.float64)
    T = len(tokens)
    h = _f(w["embed"])[tokens]
    E, F, S = MOE["n_experts"], MOE["expert_ffn"], MOE["n_shared"]
    for l in range(SH.n_layers):
        a = f32(np.stack([_rms(h[t], _f(w["attn_norm"][l]), SH.rms_eps) for t in range(T)]))
        qkv = f32(a @ _f(w["wqkv"][l]).T)
        QD = nh * (nope + rope)
        W = _f(m["wkv_b"][l]).reshape(nh, nope + vh, rank)
        lat = f32(np.stack([_rms(qkv[t, QD:QD + rank], _f(m["kv_norm"][l]), SH.rms_eps) for t in range(T)]))
        rk = f32(np.stack([_rot(qkv[t, QD + rank:], t, SH.rope_theta) for t in range(T)]))
        o = np.zeros((T, nh * vh))
        for t in range(T):
            q = qkv[t, :QD].reshape(nh, nope + rope)
            qr = f32(np.stack([_rot(q[j, nope:], t, SH.rope_theta) for j in range(nh)]))
            o[t] = ml.attend(q[:, :nope], qr, lat[:t + 1], rk[:t + 1], W[:, :nope], W[:, nope:]).reshape(-1)
        h = f32(h + f32(f32(o) @ _f(w["wo"][l]).T))
        a = f32(np.stack([_rms(h[t], _f(w["mlp_norm"][l]), SH.rms_eps) for t in range(T)]))
        if l < MLA["first_dense"]:
            gu = f32(a @ _f(w["wgate_up"][l]).T)
            act = f32(mo.silu(gu[:, :SH.ffn]) * gu[:, SH.ffn:])
            y = act @ _f(w["wdown"][l]).T
        else:
            Wgu = _f(moe["gate_up"][l]).reshape(E + S, 2, F, SH.hidden)
            Wd = _f(moe["down"][l]).reshape(SH.hidden, E + S, F).transpose(1, 0, 2)
            shared = [(Wgu[E + s, 0], Wgu[E + s, 1], Wd[E + s]) for s in range(S)]
            y = mo.moe_ffn(a, _f(moe["router"][l]), Wgu[:E, 0], Wgu[:E, 1], Wd[:E], shared, MOE["top_k"])[0]
        h = f32(h + f32(y))
    a = f32(np.stack([_rms(h[t], _f(w["final_norm"]), SH.rms_eps) for t in range(T)]))
    return a @ _f(w["lm_head"]).T


def test_forward_is_the_composition_of_its_pinned_pieces(orc):
    w, m, moe, model = _model(orc, seed=3)
    tokens = np.array([7, 0, 49, 21, 21, 3, 30], np.int32)
    cache = model.new_cache(16)
    got = model.forward(tokens, 0, cache, want="all")
    ref = _forward_numpy(w, m, moe, tokens)
    assert got.shape == ref.shape
    assert np.abs(got - ref).max() <= 2e-4 * np.abs(ref).max(), np.abs(got - ref).max()
    # every part matters at this tolerance: a changed position of one token changes the logits far more
    cache2 = model.new_cache(16)
    shifted = model.forward(tokens[1:], 0, cache2, want="all")
    assert np.abs(shifted - ref[1:]).max() > 1e-2 * np.abs(ref).max()


def test_prefill_equals_decode_token_by_token(orc):
    _, _, _, model = _model(orc, seed=4)
    tokens = np.array([5, 9, 1, 44, 17, 2], np.int32)
    c1 = model.new_cache(8)
    full = model.forward(tokens, 0, c1, want="all")
    c2 = model.new_cache(8)
    for t in range(len(tokens)):
        step = model.forward(tokens[t:t + 1], t, c2, want="last")
        assert np.abs(step - full[t]).max() <= 1e-5 * max(1.0, np.abs(full[t]).max())
    assert np.array_equal(c1[0][:, :len(tokens)], c2[0][:, :len(tokens)])


def test_bad_arguments(orc):
    _, _, _, model = _model(orc, seed=4)
    with pytest.raises(ValueError):
        model.forward(np.array([50], np.int32), 0, model.new_cache(4))      # token beyond the vocabulary
    with pytest.raises(ValueError):
        model.forward(np.array([1, 2, 3], np.int32), 2, model.new_cache(4))  # runs past the cache
