"""Pins for the oracle's elementary operators: closed forms, invariants and
brute force, each chosen so that a plausible slip (sign, index, transposed
operand, dropped term) fails."""
import math

import numpy as np
import pytest

from paper_2608_14376_b200 import synth

ONE = lambda n: synth.f32_to_bf16_bits(np.ones(n, np.float32))


def test_matmul_matches_fp64_triple_loop(orc):
    rng = np.random.default_rng(1)
    for (R, N, K) in [(1, 3, 5), (9, 17, 33), (8, 4, 64)]:
        Wb = synth.f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
        W = synth.bf16_bits_to_f32(Wb).astype(np.float64)
        X = rng.standard_normal((R, K)).astype(np.float32)
        ref = np.zeros((R, N))
        for r in range(R):
            for n in range(N):
                acc = 0.0
                for k in range(K):
                    acc += W[n, k] * float(X[r, k])
                ref[r, n] = acc
        out = orc.matmul_bf16(Wb, X)
        assert out.shape == (R, N)
        np.testing.assert_array_equal(out, ref.astype(np.float32))


def test_matmul_one_hot_rows_select_columns(orc):
    K, N = 12, 5
    W = np.zeros((N, K), np.float32)
    cols = [3, 0, 11, 7, 7]
    for n, c in enumerate(cols):
        W[n, c] = 1.0
    X = np.arange(2 * K, dtype=np.float32).reshape(2, K) + 0.5
    out = orc.matmul_bf16(synth.f32_to_bf16_bits(W), X)
    np.testing.assert_array_equal(out, X[:, cols])


def test_rmsnorm_constant_vector_closed_form(orc):
    H, c, eps = 64, 3.0, 1e-6
    g = np.linspace(0.5, 2.0, H).astype(np.float32)
    gb = synth.f32_to_bf16_bits(g)
    out = orc.rmsnorm(np.full(H, c, np.float32), gb, eps)
    want = synth.bf16_bits_to_f32(gb).astype(np.float64) * c / math.sqrt(c * c + eps)
    np.testing.assert_allclose(out, want, rtol=1e-7)


def test_rmsnorm_scale_invariance_and_unit_rms(orc):
    rng = np.random.default_rng(2)
    x = rng.standard_normal(256).astype(np.float32)
    a = orc.rmsnorm(x, ONE(256), 0.0)
    b = orc.rmsnorm(x * 8.0, ONE(256), 0.0)
    np.testing.assert_allclose(a, b, rtol=1e-6)
    assert abs(float(np.sqrt(np.mean(a.astype(np.float64) ** 2))) - 1.0) < 1e-6


def test_rmsnorm_eps_matters(orc):
    x = np.full(16, 1e-3, np.float32)
    out = orc.rmsnorm(x, ONE(16), 1e-6)
    np.testing.assert_allclose(out, 1e-3 / math.sqrt(1e-6 + 1e-6), rtol=1e-6)


def test_rope_position_zero_is_identity(orc):
    v = np.arange(64, dtype=np.float32)
    np.testing.assert_array_equal(orc.rope(v, 0, 10000.0), v)


def test_rope_known_rotation_pins_pairing_and_sign(orc):
    hd, theta = 8, 10000.0
    # unit vector on element 0: its partner is element hd/2; frequency of pair 0 is 1
    v = np.zeros(hd, np.float32); v[0] = 1.0
    out = orc.rope(v, 1, theta)
    want = np.zeros(hd); want[0] = math.cos(1.0); want[hd // 2] = math.sin(1.0)
    np.testing.assert_allclose(out, want, atol=1e-7)
    # pair 1 turns by theta^(-2/hd) per position
    v = np.zeros(hd, np.float32); v[1 + hd // 2] = 2.0
    ang = 3 * theta ** (-2.0 / hd)
    out = orc.rope(v, 3, theta)
    want = np.zeros(hd); want[1] = -2.0 * math.sin(ang); want[1 + hd // 2] = 2.0 * math.cos(ang)
    np.testing.assert_allclose(out, want, atol=1e-7)


def test_rope_preserves_norm_per_pair(orc):
    rng = np.random.default_rng(3)
    v = rng.standard_normal(128).astype(np.float32)
    for pos in (1, 17, 4095):
        out = orc.rope(v, pos, 1e6).astype(np.float64)
        pair = lambda a: a[:64] ** 2 + a[64:] ** 2
        np.testing.assert_allclose(pair(out), pair(v.astype(np.float64)), rtol=1e-5)
        assert abs(np.linalg.norm(out) - np.linalg.norm(v)) < 1e-5


def test_rope_inner_product_depends_on_relative_position(orc):
    rng = np.random.default_rng(4)
    q = rng.standard_normal(64).astype(np.float32)
    k = rng.standard_normal(64).astype(np.float32)
    d = [float(np.dot(orc.rope(q, m, 1e4).astype(np.float64), orc.rope(k, n, 1e4).astype(np.float64)))
         for (m, n) in [(5, 2), (105, 102), (40, 37)]]
    assert abs(d[0] - d[1]) < 1e-4 and abs(d[0] - d[2]) < 1e-4
    d2 = float(np.dot(orc.rope(q, 5, 1e4), orc.rope(k, 3, 1e4)))
    assert abs(d[0] - d2) > 1e-3


def test_silu_values_and_derivative(orc):
    assert orc.silu(0.0) == 0.0
    assert abs(orc.silu(30.0) - 30.0) < 1e-9
    assert abs(orc.silu(-30.0)) < 1e-9
    assert abs(orc.silu(1.0) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    z, h = 0.7, 1e-6
    sig = 1.0 / (1.0 + math.exp(-z))
    fd = (orc.silu(z + h) - orc.silu(z - h)) / (2 * h)
    assert abs(fd - (sig + z * sig * (1 - sig))) < 1e-8


def _brute_attention(q, K, V, p):
    nq, hd = q.shape
    nkv = K.shape[1]
    out = np.zeros((nq, hd))
    for j in range(nq):
        g = j // (nq // nkv)
        s = np.array([np.dot(q[j].astype(np.float64), K[t, g].astype(np.float64)) / math.sqrt(hd)
                      for t in range(p + 1)])
        e = np.exp(s)            # no max subtraction: the explicit definition
        w = e / e.sum()
        for t in range(p + 1):
            out[j] += w[t] * V[t, g].astype(np.float64)
    return out


def test_attention_matches_explicit_softmax(orc):
    rng = np.random.default_rng(5)
    nq, nkv, hd, T = 4, 2, 16, 23
    q = rng.standard_normal((nq, hd)).astype(np.float32)
    K = rng.standard_normal((T, nkv, hd)).astype(np.float32)
    V = rng.standard_normal((T, nkv, hd)).astype(np.float32)
    for p in (0, 7, T - 1):
        np.testing.assert_allclose(orc.attention(q, K, V, p), _brute_attention(q, K, V, p), rtol=2e-6, atol=1e-7)


def test_attention_is_causal_ignores_later_positions(orc):
    rng = np.random.default_rng(6)
    q = rng.standard_normal((4, 8)).astype(np.float32)
    K = rng.standard_normal((10, 2, 8)).astype(np.float32)
    V = rng.standard_normal((10, 2, 8)).astype(np.float32)
    a = orc.attention(q, K, V, 4)
    K[5:] = 1e6; V[5:] = -1e6
    np.testing.assert_array_equal(a, orc.attention(q, K, V, 4))


def test_attention_closed_forms(orc):
    rng = np.random.default_rng(7)
    nq, nkv, hd, T = 4, 2, 8, 9
    q = rng.standard_normal((nq, hd)).astype(np.float32)
    V = rng.standard_normal((T, nkv, hd)).astype(np.float32)
    # single token -> its value row, per kv group (pins the q-head -> kv-head map)
    out = orc.attention(q, np.zeros((T, nkv, hd), np.float32), V, 0)
    for j in range(nq):
        np.testing.assert_allclose(out[j], V[0, j // 2], rtol=1e-7)
    # equal keys, or q = 0 -> mean of value rows
    Keq = np.tile(rng.standard_normal((1, nkv, hd)).astype(np.float32), (T, 1, 1))
    for qq, KK in ((q, Keq), (np.zeros_like(q), rng.standard_normal((T, nkv, hd)).astype(np.float32))):
        out = orc.attention(qq, KK, V, T - 1)
        for j in range(nq):
            np.testing.assert_allclose(out[j], V[:, j // 2].astype(np.float64).mean(0), rtol=1e-6, atol=1e-7)
    # one dominant score -> that value row
    K = np.zeros((T, nkv, hd), np.float32)
    qd = np.zeros((nq, hd), np.float32); qd[:, 0] = 1.0
    K[3, :, 0] = 1e4
    out = orc.attention(qd, K, V, T - 1)
    for j in range(nq):
        np.testing.assert_allclose(out[j], V[3, j // 2], rtol=1e-6)


def test_attention_scale_is_inverse_sqrt_head_dim(orc):
    # two keys, scores differ by d/sqrt(hd): weights must be sigmoid of that
    hd = 16
    q = np.zeros((1, hd), np.float32); q[0, 0] = 2.0
    K = np.zeros((2, 1, hd), np.float32); K[1, 0, 0] = 3.0
    V = np.zeros((2, 1, hd), np.float32); V[1, 0, :] = 1.0
    out = orc.attention(q, K, V, 1)
    want = 1.0 / (1.0 + math.exp(-6.0 / math.sqrt(hd)))
    np.testing.assert_allclose(out[0], want, rtol=1e-6)
