"""GPU parity and position invariance of the Mixture-of-Experts feed-forward block against its CPU oracle."""
import numpy as np
import pytest

from oracle import moe_oracle as mo
from paper_2608_14376_b200 import synth

pytestmark = pytest.mark.gpu

# max |y - oracle| <= TOL * max |oracle|: activations enter both GEMMs as bf16 hi + lo (16 significant bits,
# relative error 2^-17 per factor), products are exact and accumulate in fp32 over at most
# (top_k + shared) * F + H terms; observed 5e-6 .. 7e-6.
TOL = 1e-4
GAP = 1e-5          # expert choices must agree where the oracle's gap between ranks top_k and top_k + 1 exceeds this


def _bf16(a):
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.asarray(a, np.float32)))


def _weights(H, E, F, S, seed):
    rng = np.random.default_rng(seed)
    NB = E + S
    return dict(router=_bf16(rng.standard_normal((E, H)) * 0.05), Wg=_bf16(rng.standard_normal((NB, F, H)) * 0.05),
                Wu=_bf16(rng.standard_normal((NB, F, H)) * 0.05), Wd=_bf16(rng.standard_normal((NB, H, F)) * 0.05))


def _device_op(corun, torch, w, H, E, K, F, S, B, renorm=False):
    NB = E + S
    gate_up = np.concatenate([np.concatenate([w["Wg"][e], w["Wu"][e]], 0) for e in range(NB)], 0)   # [(NB) * 2F, H]
    down = np.concatenate([w["Wd"][e] for e in range(NB)], 1)                                         # [H, NB * F]
    t = lambda a: torch.tensor(np.ascontiguousarray(a), dtype=torch.float32).to(torch.bfloat16).cuda().contiguous()
    return corun.MoeFfn(H, E, K, F, S, t(w["router"]), t(gate_up), t(down), B, renormalize=renorm)


@pytest.mark.parametrize("H,E,K,F,S,B,renorm", [(256, 8, 2, 128, 1, 16, False), (512, 64, 6, 192, 2, 40, False),
                                                  (128, 5, 5, 64, 0, 3, False), (256, 16, 4, 128, 1, 100, False),
                                                  (256, 32, 8, 128, 0, 24, True),
                                                  # above 64 rows the grouped form (blocks of 64 rows per expert; experts
                                                  # and shared experts with more than one block), routing weight and SwiGLU
                                                  # in the per-block GEMM's epilogue, with tiles of 96 and of 128 gate rows
                                                  # (the DeepSeek-V2-Lite expert width)
                                                  (512, 64, 6, 192, 2, 72, False), (256, 6, 2, 1408, 2, 128, False)])
def test_moe_matches_oracle_and_is_position_invariant(H, E, K, F, S, B, renorm):
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    w = _weights(H, E, F, S, seed=H + E)
    op = _device_op(corun, torch, w, H, E, K, F, S, B, renorm)
    rng = np.random.default_rng(7 * B)
    X = rng.standard_normal((B, H)).astype(np.float32)
    X[B - 1] = 0.0                                  # all router logits equal: the tie rule decides
    y, ex, pr = op.forward(torch.tensor(X).cuda())
    op.sync()
    y, ex, pr = y.cpu().numpy(), ex.cpu().numpy(), pr.cpu().numpy()
    assert list(ex[B - 1]) == list(range(K))        # ties go to the lower expert id
    shared = [(w["Wg"][E + s], w["Wu"][E + s], w["Wd"][E + s]) for s in range(S)]
    # the oracle on its own routing, and on the GPU's where a near-tie fell the other way
    Y0, ids0, _ = mo.moe_ffn(X, w["router"], w["Wg"], w["Wu"], w["Wd"], shared, K, renormalize=renorm)
    clear = []
    for b in range(B):
        _, _, p_all = mo.router(X[b], w["router"], K)
        srt = np.sort(p_all)[::-1]
        gap = srt[K - 1] - srt[K] if K < E else 1.0
        if gap > GAP and np.min(np.abs(np.diff(srt[:K]))) > GAP if K > 1 else gap > GAP:
            assert list(ex[b]) == list(ids0[b]), (b, ex[b], ids0[b])
            clear.append(b)
        assert sorted(ex[b]) == sorted(set(ex[b])) and ex[b].min() >= 0 and ex[b].max() < E
        want_p = p_all[ex[b]] / (p_all[ex[b]].sum() if renorm else 1.0)
        np.testing.assert_allclose(pr[b], want_p, atol=2e-6, rtol=2e-6)
    assert len(clear) >= B // 2
    # where the routing is clear the block's output is the oracle's, on the oracle's own routing
    assert float(np.abs(y[clear] - Y0[clear]).max() / np.abs(Y0).max()) <= TOL
    Y1, _, _ = mo.moe_ffn(X, w["router"], w["Wg"], w["Wu"], w["Wd"], shared, K, experts=ex, renormalize=renorm)
    err = float(np.abs(y - Y1).max() / np.abs(Y1).max())
    print('moe relative error', (H, E, K, F, S, B), err)
    assert err <= TOL, err

    # position invariance: the same rows at other indices among other co-tenants, byte for byte
    perm = rng.permutation(B)
    keep = perm[: max(1, B // 2)]                   # rows that are kept (moved); the others are replaced
    X2 = rng.standard_normal((B, H)).astype(np.float32) * 3.0
    X2[: len(keep)] = X[keep]
    y2, ex2, pr2 = op.forward(torch.tensor(X2).cuda())
    op.sync()
    y2, ex2, pr2 = y2.cpu().numpy(), ex2.cpu().numpy(), pr2.cpu().numpy()
    for i, r in enumerate(keep):
        assert y2[i].tobytes() == y[r].tobytes(), (i, r)
        assert ex2[i].tobytes() == ex[r].tobytes() and pr2[i].tobytes() == pr[r].tobytes()
    # and a repeat gives the same bytes
    y3, _, _ = op.forward(torch.tensor(X2).cuda())
    op.sync()
    assert y3.cpu().numpy().tobytes() == y2.tobytes()
    # up to 64 padded rows: split, router, two GEMMs, SwiGLU, read-out; above (the grouped form, where its tile widths
    # fit): split, router, grouping, gather, two grouped GEMMs, combine; else the first GEMM applies the SwiGLU itself
    assert op.launches() in (5, 6, 7)
    op.close()


def test_moe_error_paths():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_14376_b200 import corun

    w = _weights(128, 4, 64, 0, seed=3)
    with pytest.raises(corun.CorunError):           # top_k > E
        _device_op(corun, torch, w, 128, 4, 5, 64, 0, 8)
    with pytest.raises(corun.CorunError):           # B out of range
        _device_op(corun, torch, w, 128, 4, 2, 64, 0, 257)
