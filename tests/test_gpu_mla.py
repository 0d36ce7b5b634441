"""Absorbed multi-head latent attention over a paged latent cache against its oracle; independence of a row from
the other rows of the call and from where its pages lie in the pool."""
import math

import numpy as np
import pytest

from oracle import mla_oracle as ml

pytestmark = pytest.mark.gpu

PAGE = 16


def _torch():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch


def _paged(rng, caches, ctxs, dk, spare=7, fill=0.25):
    """Scatters every row's tokens over randomly chosen pages of one pool.  Returns (pool fp16 [P, 16, dk],
    block table int32 [B, max_blocks]).  Pages and positions that no row uses hold finite filler values."""
    max_blocks = max(1, max(-(-c // PAGE) for c in ctxs))
    need = sum(-(-c // PAGE) for c in ctxs)
    n_pages = need + spare
    pool = (rng.standard_normal((n_pages, PAGE, dk)) * fill).astype(np.float16)
    order = rng.permutation(n_pages)
    table = np.zeros((len(ctxs), max_blocks), np.int32)
    k = 0
    for b, c in enumerate(ctxs):
        for i in range(-(-c // PAGE)):
            pg = int(order[k]); k += 1
            table[b, i] = pg
            n = min(PAGE, c - i * PAGE)
            pool[pg, :n] = caches[b][i * PAGE:i * PAGE + n]
    return pool, table


def _case(nh, dc, dr, ctxs, seed):
    rng = np.random.default_rng(seed)
    B = len(ctxs)
    q_lat = rng.standard_normal((B, nh, dc)).astype(np.float32)
    q_rope = rng.standard_normal((B, nh, dr)).astype(np.float32)
    caches = [(rng.standard_normal((c, dc + dr)) * 0.5).astype(np.float16) for c in ctxs]
    return rng, q_lat, q_rope, caches


def _run(torch, q_lat, q_rope, pool, table, ctxs, scale):
    from paper_2608_14376_b200 import corun

    dev = lambda a: torch.tensor(a).cuda().contiguous()
    out = corun.mla_attend(dev(q_lat), dev(q_rope), dev(pool), dev(table), dev(np.array(ctxs, np.int32)), scale)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _worst(out, q_lat, q_rope, caches, ctxs, dc):
    nh = q_lat.shape[1]
    eye = np.stack([np.eye(dc)] * nh)               # W_uk = W_uv = identity: the absorbed level itself
    worst = 0.0
    for b, n in enumerate(ctxs):
        if n == 0:
            assert not out[b].any()                  # a padding row is left alone
            continue
        C = caches[b][:n, :dc].astype(np.float64)
        Rk = caches[b][:n, dc:].astype(np.float64)
        ref = ml.attend_absorbed(q_lat[b], q_rope[b], C, Rk, eye, eye)
        worst = max(worst, float(np.abs(out[b] - ref).max()))
    return worst


@pytest.mark.parametrize("nh,dc,dr", [(16, 512, 64), (4, 64, 8), (8, 128, 32), (16, 512, 24), (2, 256, 16), (1, 64, 64), (5, 128, 40)])
def test_mla_attend_matches_oracle_and_rows_are_independent(nh, dc, dr):
    torch = _torch()
    # contexts: padding row, one token, around the softmax warps' half (128), the split boundary (256), two splits, ragged pages
    ctxs = [0, 1, 127, 128, 129, 255, 256, 257, 385, 513, 700, 16]
    rng, q_lat, q_rope, caches = _case(nh, dc, dr, ctxs, seed=nh + dc)
    scale = 1.0 / math.sqrt(dc + dr)
    pool, table = _paged(rng, caches, ctxs, dc + dr)
    out = _run(torch, q_lat, q_rope, pool, table, ctxs, scale)
    # fp16 hi + lo operand pairs, fp32 accumulation chains of <= 576 and <= 128 terms on O(1) values
    worst = _worst(out, q_lat, q_rope, caches, ctxs, dc)
    assert worst <= 2e-5, worst
    # the same rows in another order, among other rows, with their pages elsewhere in a larger pool: byte-identical
    perm = [10, 2, 7, 4, 9]
    other = [300, 5, 64, 9, 0, 17, 640]
    ctx2 = [ctxs[i] for i in perm] + other
    rng2, q2, r2, c2 = _case(nh, dc, dr, ctx2, seed=99)
    for i, src in enumerate(perm):
        q2[i], r2[i], c2[i] = q_lat[src], q_rope[src], caches[src]
    pool2, table2 = _paged(rng2, c2, ctx2, dc + dr, spare=40)
    out2 = _run(torch, q2, r2, pool2, table2, ctx2, scale)
    for i, src in enumerate(perm):
        assert out2[i].tobytes() == out[src].tobytes()
    assert _worst(out2, q2, r2, c2, ctx2, dc) <= 2e-5


def test_mla_long_contexts_many_splits_and_repeatability():
    """More splits than fit one CTA's stretch, several rows per CTA and rows spread over many CTAs; twice the same bytes."""
    torch = _torch()
    nh, dc, dr = 16, 512, 64
    ctxs = [2049, 1536, 511, 4000, 3, 130]
    rng, q_lat, q_rope, caches = _case(nh, dc, dr, ctxs, seed=11)
    scale = 1.0 / math.sqrt(128 + dr)
    pool, table = _paged(rng, caches, ctxs, dc + dr)
    out = _run(torch, q_lat, q_rope, pool, table, ctxs, scale)
    again = _run(torch, q_lat, q_rope, pool, table, ctxs, scale)
    assert out.tobytes() == again.tobytes()
    nh_, eye = q_lat.shape[1], None
    worst = 0.0
    for b, n in enumerate(ctxs):
        C = caches[b][:n, :dc].astype(np.float64)
        Rk = caches[b][:n, dc:].astype(np.float64)
        # the oracle's absorbed form with identity up-projections and this scale: softmax((q_lat.C + q_rope.R) * scale).C
        s = (C @ q_lat[b].astype(np.float64).T + Rk @ q_rope[b].astype(np.float64).T) * scale      # [T, nh]
        p = np.exp(s - s.max(0)); p /= p.sum(0)
        ref = p.T @ C
        worst = max(worst, float(np.abs(out[b] - ref).max()))
    assert worst <= 2e-5, worst


def test_mla_many_rows_and_few_items():
    """More rows than one warp scans at once and more than there are CTAs (the stretches are cut inside and between
    rows by accumulated cost), padding rows in between; and a call with fewer items than CTAs."""
    torch = _torch()
    nh, dc, dr = 4, 64, 8
    rng0 = np.random.default_rng(5)
    for B, hi in ((257, 600), (3, 40)):
        ctxs = [int(c) for c in rng0.integers(0, hi, size=B)]
        ctxs[0] = 0
        ctxs[-1] = hi
        rng, q_lat, q_rope, caches = _case(nh, dc, dr, ctxs, seed=B)
        scale = 1.0 / math.sqrt(dc + dr)
        pool, table = _paged(rng, caches, ctxs, dc + dr)
        out = _run(torch, q_lat, q_rope, pool, table, ctxs, scale)
        worst = 0.0
        for b, n in enumerate(ctxs):
            if n == 0:
                assert not out[b].any()
                continue
            C = caches[b][:n, :dc].astype(np.float64)
            Rk = caches[b][:n, dc:].astype(np.float64)
            s = (C @ q_lat[b].astype(np.float64).T + Rk @ q_rope[b].astype(np.float64).T) * scale
            p = np.exp(s - s.max(0)); p /= p.sum(0)
            worst = max(worst, float(np.abs(out[b] - p.T @ C).max()))
        assert worst <= 2e-5, (B, worst)


def test_mla_context_beyond_the_block_table_is_cut():
    torch = _torch()
    nh, dc, dr, T = 8, 128, 32, 640
    rng, q_lat, q_rope, caches = _case(nh, dc, dr, [T, T], seed=3)
    scale = 1.0 / math.sqrt(dc + dr)
    pool, table = _paged(rng, caches, [T, T], dc + dr)
    full = _run(torch, q_lat, q_rope, pool, table, [T, T], scale)
    over = _run(torch, q_lat, q_rope, pool, table, [T + 100, 1 << 30], scale)
    assert over.tobytes() == full.tobytes()


def test_mla_argument_errors():
    torch = _torch()
    from paper_2608_14376_b200 import corun

    z = lambda *s: torch.zeros(s, device="cuda")
    ok = dict(pool=z(4, 16, 72).half(), table=torch.zeros((1, 2), dtype=torch.int32, device="cuda"),
              ctx=torch.ones(1, dtype=torch.int32, device="cuda"))
    with pytest.raises(corun.CorunError):            # latent width that is not 64 / 128 / 256 / 512
        corun.mla_attend(z(1, 4, 192), z(1, 4, 8), z(4, 16, 200).half(), ok["table"], ok["ctx"], 1.0)
    with pytest.raises(corun.CorunError):            # more than 16 heads
        corun.mla_attend(z(1, 17, 64), z(1, 17, 8), ok["pool"], ok["table"], ok["ctx"], 1.0)
    with pytest.raises(corun.CorunError):            # scale must be positive
        corun.mla_attend(z(1, 4, 64), z(1, 4, 8), ok["pool"], ok["table"], ok["ctx"], 0.0)
