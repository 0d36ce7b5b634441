"""Pins for the oracle's whole forward pass."""
import numpy as np
import pytest

from paper_2608_14376_b200 import synth

SMALL = synth.ModelShape(2, 64, 4, 2, 16, 96, 128, 1e-6, 10000.0)


def _model(orc, sh, w):
    return orc.Model(orc.Shape(**sh.dict()), w)


def test_matches_library_decoder_on_tiny_shape(orc):
    """The tiny-shape weights loaded into a stock fp32 Llama-style decoder
    (no QK-norm, no bias, untied head, half-split RoPE) give the same logits."""
    torch = pytest.importorskip("torch")
    tf = pytest.importorskip("transformers")
    sh = synth.TINY
    w = synth.make_weights_numpy(sh, seed=0)
    cfg = tf.LlamaConfig(vocab_size=sh.vocab, hidden_size=sh.hidden, intermediate_size=sh.ffn,
                         num_hidden_layers=sh.n_layers, num_attention_heads=sh.n_q_heads,
                         num_key_value_heads=sh.n_kv_heads, head_dim=sh.head_dim, rms_norm_eps=sh.rms_eps,
                         rope_theta=sh.rope_theta, max_position_embeddings=256, tie_word_embeddings=False,
                         attention_bias=False, mlp_bias=False, hidden_act="silu")
    cfg._attn_implementation = "eager"
    with torch.no_grad():
        m = tf.LlamaForCausalLM(cfg).to(torch.float32).eval()
        f = lambda b: torch.from_numpy(synth.bf16_bits_to_f32(b).copy())
        m.model.embed_tokens.weight.copy_(f(w["embed"]))
        m.lm_head.weight.copy_(f(w["lm_head"]))
        m.model.norm.weight.copy_(f(w["final_norm"]))
        for l, layer in enumerate(m.model.layers):
            qkv = f(w["wqkv"][l])
            layer.self_attn.q_proj.weight.copy_(qkv[:sh.q_dim])
            layer.self_attn.k_proj.weight.copy_(qkv[sh.q_dim:sh.q_dim + sh.kv_dim])
            layer.self_attn.v_proj.weight.copy_(qkv[sh.q_dim + sh.kv_dim:])
            layer.self_attn.o_proj.weight.copy_(f(w["wo"][l]))
            gu = f(w["wgate_up"][l])
            layer.mlp.gate_proj.weight.copy_(gu[:sh.ffn])
            layer.mlp.up_proj.weight.copy_(gu[sh.ffn:])
            layer.mlp.down_proj.weight.copy_(f(w["wdown"][l]))
            layer.input_layernorm.weight.copy_(f(w["attn_norm"][l]))
            layer.post_attention_layernorm.weight.copy_(f(w["mlp_norm"][l]))
        toks = synth.make_prompts(sh.vocab, [37], seed=11)[0]
        ref = m(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    model = _model(orc, sh, w)
    out = model.forward(toks, 0, model.new_cache(64), want="all")
    assert np.abs(out - ref).max() < 1e-4
    assert np.abs(ref).max() > 0.5


def test_prefill_then_decode_equals_longer_prefill(orc):
    sh = SMALL
    model = _model(orc, sh, synth.make_weights_numpy(sh, seed=3))
    toks = synth.make_prompts(sh.vocab, [21], seed=4)[0]
    full = model.forward(toks, 0, model.new_cache(32))
    c = model.new_cache(32)
    model.forward(toks[:-1], 0, c, want="none")
    step = model.forward(toks[-1:], 20, c)
    np.testing.assert_array_equal(full, step)
    c2 = model.new_cache(32)
    model.forward(toks[:9], 0, c2, want="none")
    chunked = model.forward(toks[9:], 9, c2)
    np.testing.assert_array_equal(full, chunked)


def test_row_bytes_independent_of_cotenants_padding_and_order(orc):
    sh = SMALL
    model = _model(orc, sh, synth.make_weights_numpy(sh, seed=5))
    prompts = synth.make_prompts(sh.vocab, [7, 12, 5, 9], seed=6)
    alone = model.forward(prompts[1], 0, model.new_cache(16))
    rows = [(p, 0, model.new_cache(16)) for p in prompts]
    together = orc.forward_rows(model, rows)
    np.testing.assert_array_equal(alone, together[1])
    other = synth.make_prompts(sh.vocab, [3, 12, 14], seed=99)
    rows = [(other[0], 0, model.new_cache(16)), (other[2], 0, model.new_cache(16)),
            (prompts[1], 0, model.new_cache(16))]
    np.testing.assert_array_equal(alone, orc.forward_rows(model, rows)[2])


def test_degenerate_network_closed_form(orc):
    """With Wo = Wdown = 0 every layer is the identity on the residual stream,
    so logits = Wlm * rmsnorm(E[x])."""
    sh = SMALL
    w = synth.make_weights_numpy(sh, seed=7)
    for l in range(sh.n_layers):
        w["wo"][l][:] = 0
        w["wdown"][l][:] = 0
    model = _model(orc, sh, w)
    toks = np.array([5, 77, 19], np.int32)
    out = model.forward(toks, 0, model.new_cache(8), want="all")
    E = synth.bf16_bits_to_f32(w["embed"]).astype(np.float64)
    Wlm = synth.bf16_bits_to_f32(w["lm_head"]).astype(np.float64)
    for i, t in enumerate(toks):
        x = E[t]
        a = (x / np.sqrt((x * x).mean() + sh.rms_eps)).astype(np.float32).astype(np.float64)
        np.testing.assert_allclose(out[i], Wlm @ a, rtol=1e-6, atol=1e-7)


def test_position_matters_through_rope(orc):
    sh = SMALL
    model = _model(orc, sh, synth.make_weights_numpy(sh, seed=8))
    a = model.forward([3, 4, 5], 0, model.new_cache(8))
    b = model.forward([4, 3, 5], 0, model.new_cache(8))
    assert np.abs(a - b).max() > 1e-4


def test_request_loop_is_deterministic_and_seed_bound(orc):
    sh = SMALL
    model = _model(orc, sh, synth.make_weights_numpy(sh, seed=9))
    prompt = synth.make_prompts(sh.vocab, [6], seed=10)[0]

    def run(seed):
        r = orc.Request(model, prompt, seed, temperature=0.7, top_p=0.95, max_T=16)
        return [r.prefill()] + [r.decode() for _ in range(6)]

    assert run(1000) == run(1000)
    assert run(1000) != run(1001)


def test_bad_arguments_are_rejected(orc):
    sh = SMALL
    model = _model(orc, sh, synth.make_weights_numpy(sh, seed=1))
    with pytest.raises(ValueError):
        model.forward([sh.vocab], 0, model.new_cache(4))
    with pytest.raises(ValueError):
        model.forward([1, 2, 3, 4, 5], 0, model.new_cache(4))
