"""Pins of the multi-head latent attention oracle against things other than itself (CPU)."""
import math

import numpy as np
import pytest

from oracle import mla_oracle as ml


def _case(seed, n_heads=4, d_n=8, d_r=4, d_c=16, d_v=6, T=11):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n_heads, d_n)), rng.standard_normal((n_heads, d_r)), rng.standard_normal((T, d_c)),
            rng.standard_normal((T, d_r)), rng.standard_normal((n_heads, d_n, d_c)) * 0.3,
            rng.standard_normal((n_heads, d_v, d_c)) * 0.3)


@pytest.mark.parametrize("seed", range(4))
def test_definition_equals_absorbed_form(seed):
    a = _case(seed)
    np.testing.assert_allclose(ml.attend(*a), ml.attend_absorbed(*a), rtol=1e-11, atol=1e-13)


def test_definition_equals_library_attention_on_decompressed_keys_and_values():
    torch = pytest.importorskip("torch")
    q_nope, q_rope, C, Rk, W_uk, W_uv = _case(7, T=23)
    n_heads = q_nope.shape[0]
    K = np.stack([np.concatenate([C @ W_uk[h].T, Rk], 1) for h in range(n_heads)])        # [h, T, d_n + d_r]
    V = np.stack([C @ W_uv[h].T for h in range(n_heads)])                                   # [h, T, d_v]
    Q = np.concatenate([q_nope, q_rope], 1)[:, None, :]                                      # [h, 1, d_n + d_r]
    ref = torch.nn.functional.scaled_dot_product_attention(torch.tensor(Q), torch.tensor(K), torch.tensor(V))
    np.testing.assert_allclose(ml.attend(q_nope, q_rope, C, Rk, W_uk, W_uv), ref[:, 0].numpy(), rtol=1e-10, atol=1e-12)


def test_hand_computed_two_tokens():
    """One head, d_n = d_r = d_c = d_v = 1, W_uk = 2, W_uv = 3: scores (q_n * 2 c_t + q_r * r_t) / sqrt(2)."""
    q_nope, q_rope = np.array([[1.0]]), np.array([[0.5]])
    C, Rk = np.array([[1.0], [2.0]]), np.array([[2.0], [-2.0]])
    s = [(1 * 2 * 1 + 0.5 * 2) / math.sqrt(2), (1 * 2 * 2 + 0.5 * -2) / math.sqrt(2)]     # 3/sqrt2 both
    p = [math.exp(x) / sum(math.exp(y) for y in s) for x in s]
    want = p[0] * 3 * 1.0 + p[1] * 3 * 2.0
    got = ml.attend(q_nope, q_rope, C, Rk, np.array([[[2.0]]]), np.array([[[3.0]]]))
    np.testing.assert_allclose(got, [[want]], rtol=1e-12)
    assert abs(p[0] - 0.5) < 1e-12                  # the two scores are equal: the output is the mean value, 4.5
    np.testing.assert_allclose(got, [[4.5]], rtol=1e-12)


def test_one_cached_token_returns_its_value_and_basis_change_is_invisible():
    q_nope, q_rope, C, Rk, W_uk, W_uv = _case(9, T=1)
    o = ml.attend(q_nope, q_rope, C, Rk, W_uk, W_uv)
    np.testing.assert_allclose(o, np.stack([W_uv[h] @ C[0] for h in range(q_nope.shape[0])]), rtol=1e-12)
    # an orthogonal change of basis of the latent space applied to the cache and to both up-projections
    q_nope, q_rope, C, Rk, W_uk, W_uv = _case(10)
    Qm, _ = np.linalg.qr(np.random.default_rng(3).standard_normal((C.shape[1], C.shape[1])))
    a = ml.attend_absorbed(q_nope, q_rope, C, Rk, W_uk, W_uv)
    b = ml.attend_absorbed(q_nope, q_rope, C @ Qm, Rk, W_uk @ Qm, W_uv @ Qm)
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)
